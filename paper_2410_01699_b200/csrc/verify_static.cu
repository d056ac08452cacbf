// sjd_verify_static: the isolated verification of Eqs. 1-3 for callers that must not allocate.
//
// sjd_verify takes its per-row scratch (row statistics, per-row records, ticket counters) from a
// buffer the caller allocates.  Some callers cannot do that: code running inside a region where
// device allocation is forbidden or would synchronise the device (a latency-critical serving loop,
// a host thread that does not own an allocator, a plug-in handed only input and output buffers by its
// host application).  For them the same kernel runs on a scratch area that is part of the library
// image itself: a file-scope __device__ array, present on every GPU that loads the library from load
// until exit.  Nothing is allocated or freed here, and no allocating library routine is called.
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

// Device address of the scratch on the current device.  The lookup is a host-side query of the loaded
// module (no allocation); it is repeated on every call, so the address always belongs to the context
// that is current now (a cached one would go stale after cudaDeviceReset).
int static_scratch(void **out) {
  void *p = nullptr;
  SJD_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
  if (!p) return SJD_ERR_CUDA;
  *out = p;
  return SJD_OK;
}

}  // namespace

int verify_isolated(int batch, int window, int vocab, int logits_dtype, const void *logits_cur, const void *logits_prev,
                    const int32_t *draft, const int32_t *q_kind, const int32_t *base_pos, const sjd_sample_cfg *sample,
                    uint32_t step, const sjd_step_out *out, void *scratch, cudaStream_t stream);   // api.cu
}  // namespace sjd

using namespace sjd;

extern "C" int sjd_verify_static(int batch, int window, int vocab, int logits_dtype, const void *logits_cur,
                                 const void *logits_prev, const int32_t *draft, const int32_t *q_kind,
                                 const int32_t *base_pos, const sjd_sample_cfg *sample, uint32_t step,
                                 const sjd_step_out *out, void *cuda_stream) {
  if (batch >= 1 && window >= 1 && window <= 64 &&
      (batch > kStaticMaxBatch || (long)batch * window > kStaticMaxRows))
    return SJD_ERR_CAPACITY;
  void *scratch = nullptr;
  const int rc = static_scratch(&scratch);
  if (rc != SJD_OK) return rc;
  // the shared helper checks the arguments, clears the ticket counters (the array keeps whatever the
  // previous call left) and launches the kernel
  return verify_isolated(batch, window, vocab, logits_dtype, logits_cur, logits_prev, draft, q_kind, base_pos, sample,
                         step, out, scratch, (cudaStream_t)cuda_stream);
}
