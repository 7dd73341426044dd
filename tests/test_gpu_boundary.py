"""Error behaviour of the C ABI on a GPU: every rejected call launches nothing and changes no state."""
import numpy as np
import pytest

from edgefm_synth import CONFIGS
from helpers import Pair

pytestmark = pytest.mark.gpu
TINY = CONFIGS["tiny"]


def _shape(cfg, **kw):
    d = dict(n_layers=cfg.n_layers, hidden=cfg.hidden, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
             head_dim=cfg.head_dim, ffn=cfg.ffn, vocab=cfg.vocab, rms_eps=cfg.rms_eps, rope_theta=cfg.rope_theta,
             qkv_bias=int(cfg.qkv_bias))
    d.update(kw)
    return d


def test_create_rejects_bad_shapes_and_pointers():
    from paper_2604_27476_b200 import EdgefmError, Status, edgefm_create
    pair = Pair(TINY, cache_len=0, max_context=4)
    try:
        bad = [dict(head_dim=48), dict(hidden=100), dict(ffn=7), dict(n_q_heads=3), dict(n_q_heads=18, n_kv_heads=2),
               dict(n_layers=0), dict(vocab=0), dict(rope_theta=0.0)]
        for kw in bad:
            with pytest.raises(EdgefmError) as ei:
                edgefm_create(_shape(TINY, **kw), pair.ptrs, 8)
            assert ei.value.status == Status.ERR_BAD_SHAPE, kw
        with pytest.raises(EdgefmError) as ei:
            edgefm_create(_shape(TINY), pair.ptrs, 0)
        assert ei.value.status == Status.ERR_INVALID_ARG
        ptrs = dict(pair.ptrs, embed=None)
        with pytest.raises(EdgefmError) as ei:
            edgefm_create(_shape(TINY), ptrs, 8)
        assert ei.value.status == Status.ERR_INVALID_ARG
        ptrs = dict(pair.ptrs, lm_head=pair.ptrs["lm_head"] + 2)            # misaligned
        with pytest.raises(EdgefmError) as ei:
            edgefm_create(_shape(TINY), ptrs, 8)
        assert ei.value.status == Status.ERR_INVALID_ARG
        layers = [dict(l) for l in pair.ptrs["layers"]]
        layers[1]["w_down"] = None
        with pytest.raises(EdgefmError) as ei:
            edgefm_create(_shape(TINY), dict(pair.ptrs, layers=layers), 8)
        assert ei.value.status == Status.ERR_INVALID_ARG
        with pytest.raises(EdgefmError) as ei:                                  # bias requested but missing
            edgefm_create(_shape(TINY, qkv_bias=1), pair.ptrs, 8)
        assert ei.value.status == Status.ERR_INVALID_ARG
    finally:
        pair.close()


def test_step_and_prefill_errors_change_nothing():
    import torch
    from paper_2604_27476_b200 import EdgefmError, Status
    pair = Pair(TINY, cache_len=2, max_context=4)
    try:
        ctx = pair.ctx
        for tok, pos in ((TINY.vocab, 0), (-2, 0), (0, -2), (-1, 0)):            # -1 before any step
            with pytest.raises(EdgefmError) as ei:
                ctx.step(tok, pos)
            assert ei.value.status == Status.ERR_INVALID_ARG
        assert ctx.cur_len == 2
        ctx.step(1, 2); ctx.step(-1, -1)
        assert ctx.cur_len == 4
        torch.cuda.synchronize()
        k0, v0 = [t.clone() for t in ctx.export_kv()]
        logits0 = ctx.logits.clone()
        with pytest.raises(EdgefmError) as ei:
            ctx.step(1, 4)                                                     # full cache: nothing is launched
        assert ei.value.status == Status.ERR_CONTEXT_FULL
        big = torch.zeros((TINY.n_layers, TINY.n_kv_heads, 5, TINY.head_dim), dtype=torch.int16, device="cuda")
        with pytest.raises(EdgefmError) as ei:
            ctx.prefill_kv(big, big)
        assert ei.value.status == Status.ERR_CONTEXT_FULL
        torch.cuda.synchronize()
        k1, v1 = ctx.export_kv()
        assert torch.equal(k0, k1) and torch.equal(v0, v1) and torch.equal(logits0, ctx.logits) and ctx.cur_len == 4
        ctx.reset()
        assert ctx.cur_len == 0
        ctx.step(3, 0)                                                         # usable again after reset
        torch.cuda.synchronize()
        assert ctx.cur_len == 1 and bool(torch.isfinite(ctx.logits).all())
    finally:
        pair.close()


def test_unaligned_strided_prefill_takes_the_scalar_path():
    import torch
    cfg = TINY
    pair = Pair(cfg, cache_len=0, max_context=16)
    try:
        L, g, d = cfg.n_layers, cfg.n_kv_heads, cfg.head_dim
        base = torch.randint(-3000, 3000, (L, g, 9, d + 3), dtype=torch.int16, device="cuda")
        k = base[:, :, :, 1:d + 1]                                             # odd element offset, stride_pos = d+3
        pair.ctx.prefill_kv(k, k)
        kc, vc = pair.ctx.export_kv()
        torch.cuda.synchronize()
        assert torch.equal(kc[:, :, :9], k) and torch.equal(vc[:, :, :9], k) and pair.ctx.cur_len == 9
    finally:
        pair.close()
