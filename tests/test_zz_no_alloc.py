"""edgefm_decode_step_static: the decode step for callers that cannot allocate device memory (code inside
another framework's fixed memory plan, processes living off a memory pool they do not own, threads that cannot
take cudaMalloc's implicit synchronisation).  Its work buffers are a fixed array inside the library, the KV cache
is the caller's.  Checked here against edgefm_decode_step and against the CPU oracle on the same inputs, two steps in a
row; the second call reuses the scratch array with the first call's contents still in it.

The file name makes pytest collect it last, so a run that stops at the first failure has run everything else."""
import numpy as np
import pytest

from edgefm_synth import CONFIGS, first_token
from helpers import LOGIT_MAX_ABS, LOGIT_REL_L2, Pair, compare_logits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("variant", ["tiny", "bias_long_rows", "long_context_build"])
def test_static_scratch_step_matches_context_step_twice(variant):
    import torch
    from paper_2604_27476_b200 import edgefm_decode_step_static, edgefm_sync_status
    from helpers import assert_logits_close
    cfg = CONFIGS["tiny"]
    if variant == "bias_long_rows":   # K slices, several tiles per warp, biases, many attention chunks
        cfg = cfg.with_(hidden=512, ffn=6144, vocab=20000, n_layers=3, qkv_bias=True, cache_len=700)
    T0, Tmax = cfg.cache_len, cfg.cache_len + 4
    if variant == "long_context_build":   # max_context > 8192 selects the other build of the kernel
        T0, Tmax = 300, 8300
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
            oracle_logits, oracle_next = pair.oracle.step(tok, pos)     # the CPU oracle, directly
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
            assert_logits_close(got, oracle_logits, f"static step {step} against the oracle")
            edgefm_sync_status(None, stream)                                      # the static path's own status word: no expired wait
            tok, pos, cur = ref_next, pos + 1, cur + 1
    finally:
        pair.close()


def test_static_step_interleaved_with_contexts_of_other_shapes():
    """Two live contexts of different shapes and static calls of a third shape step alternately: they select the same
    kernel instantiation with different dynamic shared-memory sizes, and none may disturb the others."""
    import torch
    from paper_2604_27476_b200 import edgefm_decode_step_static
    from helpers import assert_logits_close
    base = CONFIGS["tiny"]
    cfgs = [base, base.with_(hidden=512, ffn=1536, vocab=5000, qkv_bias=True), base.with_(hidden=384, ffn=2048, vocab=3000, n_layers=3)]
    pairs = [Pair(c, cache_len=40 + 10 * i, max_context=64 + 10 * i) for i, c in enumerate(cfgs)]
    try:
        stream = torch.cuda.current_stream().cuda_stream
        c3 = cfgs[2]
        shape3 = dict(n_layers=c3.n_layers, hidden=c3.hidden, n_q_heads=c3.n_q_heads, n_kv_heads=c3.n_kv_heads, head_dim=c3.head_dim,
                      ffn=c3.ffn, vocab=c3.vocab, rms_eps=c3.rms_eps, rope_theta=c3.rope_theta, qkv_bias=int(c3.qkv_bias))
        k3, v3 = [t.clone() for t in pairs[2].ctx.export_kv()]
        logits3 = torch.empty(c3.vocab, device="cuda")
        toks = [first_token(c) for c in cfgs]
        for s in range(3):
            refs = [p.oracle.step(toks[i], p.T0 + s) for i, p in enumerate(pairs)]
            pairs[0].ctx.step(toks[0], pairs[0].T0 + s)
            edgefm_decode_step_static(shape3, pairs[2].ptrs, k3.data_ptr(), v3.data_ptr(), pairs[2].max_context, pairs[2].T0 + s, toks[2],
                                      pairs[2].T0 + s, stream, logits3.data_ptr(), None)
            pairs[1].ctx.step(toks[1], pairs[1].T0 + s)
            torch.cuda.synchronize()
            assert_logits_close(pairs[0].ctx.logits.cpu().numpy(), refs[0][0], f"context A step {s}")
            assert_logits_close(pairs[1].ctx.logits.cpu().numpy(), refs[1][0], f"context B step {s}")
            assert_logits_close(logits3.cpu().numpy(), refs[2][0], f"static call step {s}")
            toks = [r[1] for r in refs]
    finally:
        for p in pairs:
            p.close()


def test_static_step_refuses_a_capturing_stream():
    """The call copies from host memory of the call itself; recorded into a capture that would be replayed from freed memory.
    It must therefore refuse a stream in capture mode before enqueuing anything."""
    import torch
    from paper_2604_27476_b200 import EdgefmError, Status, edgefm_decode_step_static
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, cache_len=8, max_context=16)
    try:
        shape = dict(n_layers=cfg.n_layers, hidden=cfg.hidden, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads, head_dim=cfg.head_dim,
                     ffn=cfg.ffn, vocab=cfg.vocab, rms_eps=cfg.rms_eps, rope_theta=cfg.rope_theta, qkv_bias=0)
        k, v = pair.ctx.export_kv()
        side = torch.cuda.Stream()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            g.capture_begin()
            try:
                with pytest.raises(EdgefmError) as ei:
                    edgefm_decode_step_static(shape, pair.ptrs, k.data_ptr(), v.data_ptr(), 16, 8, 1, 8, side.cuda_stream)
                assert ei.value.status == Status.ERR_INVALID_ARG and "captured" in str(ei.value)
            finally:
                g.capture_end()                                    # an empty graph: nothing was recorded
        torch.cuda.synchronize()
        edgefm_decode_step_static(shape, pair.ptrs, k.data_ptr(), v.data_ptr(), 16, 8, 1, 8, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()                                   # and the same call outside a capture runs
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
