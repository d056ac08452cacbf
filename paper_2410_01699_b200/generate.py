"""Whole-sequence generation on top of the step interface (Algorithm 1 from the caller's side).

    tokens, counts, steps = generate(ctx, prompt, sample)

Every iteration of the method (forward pass, verification, resampling, window slide) runs inside sjd_step;
this loop only enqueues iterations and looks at the per-image DONE flags every `check_every` iterations, so the
device is never idle waiting for the host: at most check_every - 1 iterations run after the last image has
finished, and a finished image takes no part in them (its window is empty).  Nothing here touches a token.
"""
from __future__ import annotations

import torch

from . import binding as B


def generate(ctx: B.Context, prompt: torch.Tensor, sample, prompt_lens=None, check_every: int = 8,
             max_steps: int | None = None):
    """prompt: int32 cuda tensor [B][P] (2 rows per image under guidance: conditional, unconditional).
    Returns (tokens int32 [images][max_seq] on the device, counts int32 [images], iterations run): row i of
    tokens holds image i's prompt followed by its sample.n_generate generated tokens."""
    if prompt_lens is None:
        ctx.prefill(prompt, sample)
    else:
        ctx.prefill_ragged(prompt, prompt_lens, sample)
    images = ctx.batch // 2 if float(sample.guidance) != 0.0 else ctx.batch
    out = B.StepOut(images, ctx.window, device=ctx.device)
    limit = int(sample.n_generate) if max_steps is None else int(max_steps)   # an iteration fixes at least one token
    steps = 0
    while steps < limit:
        n = min(check_every, limit - steps)
        for _ in range(n):
            ctx.step(out)
        steps += n
        flags = out.flags.cpu()
        if bool(((flags & B.SJD_FLAG_DONE) != 0).all()):
            break
    status = ctx.device_status()
    if status != B.SJD_OK:
        raise B.SJDError(status, "generate")
    tokens, counts = ctx.get_tokens()
    return tokens, counts, steps
