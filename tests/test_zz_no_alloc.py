"""edgefm_decode_step_static: the decode step for callers that cannot allocate device memory (code inside
another framework's fixed memory plan, processes living off a memory pool they do not own, threads that cannot
take cudaMalloc's implicit synchronisation).  Its work buffers are a fixed array inside the library, the KV cache
is the caller's.  Checked here against edgefm_decode_step on the same inputs, two steps in a row; the second
call reuses the scratch array with the first call's contents still in it.

The file name makes pytest collect it last, so a run that stops at the first failure has run everything else."""
import numpy as np
import pytest

from edgefm_synth import CONFIGS, first_token
from helpers import LOGIT_MAX_ABS, LOGIT_REL_L2, Pair, compare_logits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("variant", ["tiny", "bias_long_rows"])
def test_static_scratch_step_matches_context_step_twice(variant):
    import torch
    from paper_2604_27476_b200 import edgefm_decode_step_static
    cfg = CONFIGS["tiny"]
    if variant == "bias_long_rows":   # K slices, several tiles per warp, biases, many attention chunks
        cfg = cfg.with_(hidden=512, ffn=6144, vocab=20000, n_layers=3, qkv_bias=True, cache_len=700)
    T0, Tmax = cfg.cache_len, cfg.cache_len + 4
    pair = Pair(cfg, cache_len=T0, max_context=Tmax)
    try:
        shape = dict(n_layers=cfg.n_layers, hidden=cfg.hidden, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                     head_dim=cfg.head_dim, ffn=cfg.ffn, vocab=cfg.vocab, rms_eps=cfg.rms_eps, rope_theta=cfg.rope_theta,
                     qkv_bias=int(cfg.qkv_bias))
        stream = torch.cuda.current_stream().cuda_stream
        # the caller-owned cache of the static path starts as a copy of the context's cache
        k_own, v_own = [t.clone() for t in pair.ctx.export_kv()]
        logits = torch.full((cfg.vocab,), float("nan"), device="cuda")
        nxt = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        tok, pos, cur = first_token(cfg), cfg.first_position, T0
        for step in range(2):
            pair.ctx.step(tok, pos)                                   # existing entry point
            torch.cuda.synchronize()
            ref_logits = pair.ctx.logits.cpu().numpy().copy()
            ref_next = int(pair.ctx.next_token.item())
            k_ref, v_ref = pair.ctx.export_kv()
            logits.fill_(float("nan")); nxt.fill_(-7)
            edgefm_decode_step_static(shape, pair.ptrs, k_own.data_ptr(), v_own.data_ptr(), Tmax, cur, tok, pos, stream,
                                      logits.data_ptr(), nxt.data_ptr())
            torch.cuda.synchronize()
            got = logits.cpu().numpy()
            assert np.isfinite(got).all()
            max_abs, rel_l2 = compare_logits(got, ref_logits)
            assert max_abs <= LOGIT_MAX_ABS and rel_l2 <= LOGIT_REL_L2, (step, max_abs, rel_l2)
            assert int(nxt.item()) == ref_next
            assert torch.equal(k_own, k_ref) and torch.equal(v_own, v_ref)        # same row appended, rest untouched
            tok, pos, cur = ref_next, pos + 1, cur + 1
    finally:
        pair.close()


def test_static_scratch_step_rejects_oversized_and_bad_arguments():
    import torch
    from paper_2604_27476_b200 import EdgefmError, Status, edgefm_decode_step_static
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, cache_len=0, max_context=4)
    try:
        shape = dict(n_layers=cfg.n_layers, hidden=cfg.hidden, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                     head_dim=cfg.head_dim, ffn=cfg.ffn, vocab=cfg.vocab, rms_eps=cfg.rms_eps, rope_theta=cfg.rope_theta,
                     qkv_bias=0)
        k, v = pair.ctx.export_kv()
        torch.cuda.synchronize()
        args = (k.data_ptr(), v.data_ptr(), 4)
        with pytest.raises(EdgefmError) as ei:     # beyond what the fixed scratch array is laid out for: nothing is launched
            edgefm_decode_step_static(dict(shape, n_layers=97), pair.ptrs, *args, 0, 1, 0)
        assert ei.value.status == Status.ERR_BAD_SHAPE and "at most 96 layers" in str(ei.value)
        with pytest.raises(EdgefmError) as ei:
            edgefm_decode_step_static(shape, pair.ptrs, *args, 4, 1, 0)        # cache full
        assert ei.value.status == Status.ERR_CONTEXT_FULL
        with pytest.raises(EdgefmError) as ei:
            edgefm_decode_step_static(shape, pair.ptrs, *args, 0, -1, 0)       # token must be explicit
        assert ei.value.status == Status.ERR_INVALID_ARG
        with pytest.raises(EdgefmError) as ei:
            edgefm_decode_step_static(shape, pair.ptrs, None, v.data_ptr(), 4, 0, 1, 0)
        assert ei.value.status == Status.ERR_INVALID_ARG
    finally:
        pair.close()
