"""Fixed-prefix cache reuse (Sec. 3.9, Eq. 5: KV = Concat(KV_p, KV_u)) through edgefm_append_kv.

The oracle side is the plain definition: its cache is loaded with the concatenated arrays.  The CUDA side keeps the
prefix slots and copies only the suffix behind them.
"""
import numpy as np
import pytest

from edgefm_synth import CONFIGS, GLOBAL_SEED, first_token, make_kv
from helpers import Pair, assert_logits_close

pytestmark = pytest.mark.gpu

PREFIX = 96


def _dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()


def _oracle_logits(pair, k, v, tok, pos):
    """One oracle step over a cache holding exactly k, v."""
    from oracle import OracleModel
    o = OracleModel(pair.cfg, pair.weights, pair.max_context)
    try:
        o.load_kv(np.ascontiguousarray(k), np.ascontiguousarray(v))
        return o.step(tok, pos)
    finally:
        o.close()


def test_prefix_plus_suffix_equals_whole_prefill():
    import torch
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, max_context=cfg.cache_len + 8)          # its context was prefilled with all 128 positions
    try:
        tok, pos = first_token(cfg), cfg.first_position
        pair.ctx.step(tok, pos)
        torch.cuda.synchronize()
        whole = pair.ctx.logits.cpu().numpy().copy()
        # same cache built as prefix + suffix
        pair.ctx.prefill_kv(pair.kd[:, :, :PREFIX], pair.vd[:, :, :PREFIX])
        assert pair.ctx.cur_len == PREFIX
        pair.ctx.append_kv(PREFIX, pair.kd[:, :, PREFIX:], pair.vd[:, :, PREFIX:])   # strided views of the device arrays
        assert pair.ctx.cur_len == cfg.cache_len
        pair.ctx.step(tok, pos)
        torch.cuda.synchronize()
        assert np.array_equal(pair.ctx.logits.cpu().numpy(), whole)                    # same bits as one prefill
        ref, _ = pair.oracle.step(tok, pos)
        assert_logits_close(whole, ref, "prefix + suffix")
    finally:
        pair.close()


def test_prefix_survives_requests():
    """Request 1 decodes a few tokens; request 2 re-uses the first PREFIX slots with another suffix; request 3 uses the
    bare prefix.  Each must match the oracle run on the concatenated cache."""
    import torch
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, max_context=cfg.cache_len + 8)
    try:
        tok, pos = first_token(cfg), cfg.first_position
        for s in range(4):                                    # request 1: the cache grows to 132 slots
            pair.ctx.step(tok if s == 0 else -1, pos + s if s == 0 else -1)
        torch.cuda.synchronize()
        assert pair.ctx.cur_len == cfg.cache_len + 4
        k2, v2 = make_kv(cfg, GLOBAL_SEED + 1, 20)            # request 2: a different 20-position suffix
        pair.ctx.append_kv(PREFIX, _dev(k2), _dev(v2))
        assert pair.ctx.cur_len == PREFIX + 20
        pair.ctx.step(tok, PREFIX + 20)
        torch.cuda.synchronize()
        kc = np.concatenate([pair.k[:, :, :PREFIX], k2], axis=2)
        vc = np.concatenate([pair.v[:, :, :PREFIX], v2], axis=2)
        ref, ref_next = _oracle_logits(pair, kc, vc, tok, PREFIX + 20)
        assert_logits_close(pair.ctx.logits.cpu().numpy(), ref, "re-used prefix + new suffix")
        pair.ctx.append_kv(PREFIX)                            # request 3: truncate to the prefix, no suffix
        assert pair.ctx.cur_len == PREFIX
        pair.ctx.step(tok, -1)                                # default position = cache length
        torch.cuda.synchronize()
        ref, _ = _oracle_logits(pair, pair.k[:, :, :PREFIX], pair.v[:, :, :PREFIX], tok, PREFIX)
        assert_logits_close(pair.ctx.logits.cpu().numpy(), ref, "bare prefix")
    finally:
        pair.close()


def test_append_rejects_holes_and_overflow():
    import torch
    from paper_2604_27476_b200 import EdgefmError, Status
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, max_context=cfg.cache_len + 8)
    try:
        k_before, v_before = pair.ctx.export_kv()
        torch.cuda.synchronize()
        with pytest.raises(EdgefmError) as e:
            pair.ctx.append_kv(cfg.cache_len + 1, pair.kd[:, :, :2], pair.vd[:, :, :2])     # would leave a hole
        assert e.value.status == Status.ERR_INVALID_ARG
        with pytest.raises(EdgefmError) as e:
            pair.ctx.append_kv(cfg.cache_len, pair.kd[:, :, :9], pair.vd[:, :, :9])         # 128 + 9 > 136
        assert e.value.status == Status.ERR_CONTEXT_FULL
        with pytest.raises(EdgefmError):
            pair.ctx.append_kv(-1)
        assert pair.ctx.cur_len == cfg.cache_len
        k_after, v_after = pair.ctx.export_kv()
        torch.cuda.synchronize()
        assert torch.equal(k_before, k_after) and torch.equal(v_before, v_after)
    finally:
        pair.close()
