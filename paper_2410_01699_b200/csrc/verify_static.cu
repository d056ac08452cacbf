// sjd_verify_static: the isolated verification of Eqs. 1-3 for callers that must not allocate.
//
// sjd_verify takes its per-row scratch (row statistics, per-row records, ticket counters) from a
// buffer the caller allocates.  Some callers cannot do that: code running inside a region where
// device allocation is forbidden or would synchronise the device (a latency-critical serving loop,
// a host thread that does not own an allocator, a plug-in handed only input and output buffers by its
// host application).  For them the same kernel runs on a scratch area that is part of the library
// image itself: a file-scope __device__ array, present on every GPU that loads the library from load
// until exit.  Nothing is allocated or freed here, and no allocating library routine is called.
#include <string.h>

#include <mutex>

#include "common.cuh"

namespace sjd {
namespace {

constexpr int kStaticMaxRows = SJD_VERIFY_STATIC_MAX_ROWS;    // batch * window
constexpr int kStaticMaxBatch = SJD_VERIFY_STATIC_MAX_BATCH;
constexpr size_t kStaticBytes =
    ((size_t)kStaticMaxRows * (2 * sizeof(RowStats) + sizeof(RowOut)) + (kStaticMaxBatch + 1) * sizeof(int32_t) + 255) /
    256 * 256;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress, never an
// address a kernel could use.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void *g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch on the current device, looked up once per device.
int static_scratch(void **out) {
  int dev = -1;
  SJD_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return SJD_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    void *p = nullptr;
    SJD_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
    if (!p) return SJD_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return SJD_OK;
}

}  // namespace
}  // namespace sjd

using namespace sjd;

extern "C" int sjd_verify_static(int batch, int window, int vocab, int logits_dtype, const void *logits_cur,
                                 const void *logits_prev, const int32_t *draft, const int32_t *q_kind,
                                 const int32_t *base_pos, const sjd_sample_cfg *sample, uint32_t step,
                                 const sjd_step_out *out, void *cuda_stream) {
  if (batch < 1 || window < 1 || vocab < 1 || !logits_cur || !draft || !sample || !out) return SJD_ERR_BAD_ARG;
  if (!logits_prev && !q_kind) return SJD_ERR_BAD_ARG;
  if (logits_dtype != SJD_F32 && logits_dtype != SJD_BF16) return SJD_ERR_UNSUPPORTED;
  if (window > 64) return SJD_ERR_CAPACITY;
  if (batch > kStaticMaxBatch || (long)batch * window > kStaticMaxRows) return SJD_ERR_CAPACITY;
  if (!(sample->temperature > 0.0f) || sample->top_k < 1 || sample->seq_base < 0) return SJD_ERR_BAD_ARG;
  void *scratch = nullptr;
  const int rc = static_scratch(&scratch);
  if (rc != SJD_OK) return rc;
  cudaStream_t stream = (cudaStream_t)cuda_stream;

  const size_t rows = (size_t)batch * window;
  char *w = (char *)scratch;
  VerifyParams p;
  memset(&p, 0, sizeof(p));
  p.logits[0] = logits_cur;
  p.logits[1] = logits_prev ? logits_prev : logits_cur;
  p.stats[0] = (RowStats *)w;
  p.stats[1] = (RowStats *)(w + rows * sizeof(RowStats));
  p.row_out = (RowOut *)(w + 2 * rows * sizeof(RowStats));
  p.seq_counter = (int32_t *)(w + 2 * rows * sizeof(RowStats) + rows * sizeof(RowOut));
  p.done_counter = p.seq_counter + batch;
  // the array keeps whatever the previous call left: the ticket counters must start at zero
  SJD_CUDA(cudaMemsetAsync(p.seq_counter, 0, ((size_t)batch + 1) * sizeof(int32_t), stream));
  p.draft = draft;
  p.q_kind = q_kind;
  p.base_pos = base_pos;
  p.step = step;
  p.B = batch;
  p.W = window;
  p.V = vocab;
  p.temperature = sample->temperature;
  p.top_k = sample->top_k;
  p.seed_lo = (uint32_t)(sample->seed & 0xFFFFFFFFull);
  p.seed_hi = (uint32_t)(sample->seed >> 32);
  p.seq_base = (uint32_t)sample->seq_base;
  p.e2e = 0;
  p.out = *out;
  return launch_verify(p, logits_dtype, stream);
}
