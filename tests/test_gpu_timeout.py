"""The bounded device-side waits of the step kernel, driven to expiry without any fault: the grid barrier is told to
expect one arrival more than there are CTAs and the bound is shortened to 2 ms, so the first barrier of the next step
gives up.  The kernel must return, the status must read EDGEFM_ERR_TIMEOUT, the context must still be destroyable, and a
fresh context on the same weights must work."""
import time

import pytest

from edgefm_synth import CONFIGS, first_token
from helpers import Pair, assert_logits_close

pytestmark = pytest.mark.gpu


def test_grid_barrier_wait_expires_and_is_reported():
    import torch
    from paper_2604_27476_b200 import (DecodeContext, EdgefmError, Status, edgefm_debug_set_wait_limit, edgefm_sync_status)
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, max_context=cfg.cache_len + 8)
    try:
        stream = torch.cuda.current_stream().cuda_stream
        tok, pos = first_token(cfg), cfg.first_position
        ref, nxt = pair.oracle.step(tok, pos)
        pair.ctx.step(tok, pos)                                   # a normal step first
        edgefm_sync_status(pair.ctx.handle, stream)
        assert_logits_close(pair.ctx.logits.cpu().numpy(), ref, "before")
        edgefm_debug_set_wait_limit(pair.ctx.handle, 2_000_000, 1)    # 2 ms; the barrier now waits for a CTA that does not exist
        t0 = time.perf_counter()
        pair.ctx.step(nxt, pos + 1)
        with pytest.raises(EdgefmError) as ei:
            edgefm_sync_status(pair.ctx.handle, stream)
        dt = time.perf_counter() - t0
        assert ei.value.status == Status.ERR_TIMEOUT
        assert dt < 2.0                                            # the kernel returned by itself, well inside a second
        with pytest.raises(EdgefmError):                           # limits are validated
            edgefm_debug_set_wait_limit(pair.ctx.handle, 10, 0)
        # the CUDA context is intact: a fresh edgefm context on the same weights computes the right answer
        other = DecodeContext(cfg, pair.ptrs, cfg.cache_len + 8)
        other.prefill_kv(pair.kd, pair.vd)
        other.step(tok, pos)
        torch.cuda.synchronize()
        assert_logits_close(other.logits.cpu().numpy(), ref, "fresh context after the expired wait")
        other.close()
    finally:
        pair.close()                                               # destroying the timed-out context succeeds


def test_prefill_contraction_wait_expires_and_is_reported():
    """The same for the contractions of edgefm_prefill: their stage barriers are told to expect an arrival nobody makes and
    the bound is shortened to 2^16 polls; every contraction gives up at its first wait, drains and returns."""
    import numpy as np
    import torch
    from paper_2604_27476_b200 import DecodeContext, EdgefmError, Status, edgefm_debug_set_prefill_wait, edgefm_sync_status
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, cache_len=4, max_context=64)
    try:
        stream = torch.cuda.current_stream().cuda_stream
        toks = np.random.default_rng(3).integers(0, cfg.vocab, 40).tolist()
        for i, t in enumerate(toks):
            ref, _ = pair.oracle.step(t, 4 + i)
        with pytest.raises(EdgefmError):                           # limits are validated
            edgefm_debug_set_prefill_wait(pair.ctx.handle, 10, 0)
        edgefm_debug_set_prefill_wait(pair.ctx.handle, 1 << 16, 1)
        t0 = time.perf_counter()
        pair.ctx.prefill(toks, 4)
        with pytest.raises(EdgefmError) as ei:
            edgefm_sync_status(pair.ctx.handle, stream)
        dt = time.perf_counter() - t0
        assert ei.value.status == Status.ERR_TIMEOUT
        assert dt < 5.0                                            # five contractions, each gave up within milliseconds
        # the CUDA context is intact: a fresh edgefm context on the same weights prefills the same prompt correctly
        other = DecodeContext(cfg, pair.ptrs, 64)
        other.prefill_kv(pair.kd, pair.vd)
        other.prefill(toks, 4)
        torch.cuda.synchronize()
        other.sync_status()
        assert_logits_close(other.logits.cpu().numpy(), ref, "fresh context after the expired waits")
        other.close()
    finally:
        pair.close()
