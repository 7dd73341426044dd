"""Compressed KV cache (Sec. 3.9 of the paper: KV~ = C(KV), reconstruction on demand; reading: 8-bit codes and one fp32
scale per cached row): the CUDA path against the oracle with the same cache format.

The codes are integers decided by floating-point values, and the two sides decide them in the same precision (fp32) from
inputs that differ in the last bits (the CUDA path sums in fp32, the oracle in fp64): rows given to prefill are bf16 and
must compress to identical codes; a row appended by a step may differ by one code in a few places."""
import numpy as np
import pytest

from edgefm_synth import CONFIGS, first_token
from helpers import Pair, assert_logits_close, top2_margin, TOKEN_MARGIN

pytestmark = pytest.mark.gpu


def _shapes():
    base = CONFIGS["tiny"]
    return {
        "tiny_d64": (base, 128, 140),
        "d128_bias_gqa4": (base.with_(hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn=1536, vocab=3000, n_layers=3, qkv_bias=True), 300, 320),
        "long_ragged_chunks": (base.with_(hidden=384, n_q_heads=6, n_kv_heads=1, head_dim=128, ffn=1024, vocab=2000), 9001, 9010),
        "empty_cache": (base, 0, 6),
        # the size and cache length bench.py --config qwen2.5-7b-32k --kv-format int8 times (two steps)
        "qwen2.5-7b-32k_full_size": (CONFIGS["qwen2.5-7b-32k"], CONFIGS["qwen2.5-7b-32k"].cache_len, CONFIGS["qwen2.5-7b-32k"].cache_len + 2),
    }


@pytest.mark.parametrize("name", list(_shapes()))
def test_steps_with_compressed_cache_match_oracle(name):
    import torch
    cfg, T0, Tmax = _shapes()[name]
    pair = Pair(cfg, cache_len=T0, max_context=Tmax, kv_format="int8")
    try:
        # the given rows compress to the oracle's codes and scales exactly
        k8, v8, ks, vs = [t.cpu().numpy() for t in pair.ctx.export_kv_int8()]
        ok8, ov8, oks, ovs = pair.oracle.export_kv_q8()
        assert np.array_equal(k8, ok8) and np.array_equal(v8, ov8) and np.array_equal(ks, oks) and np.array_equal(vs, ovs)
        tok, pos = first_token(cfg), T0 + 3
        steps = min(5, Tmax - T0)
        for s in range(steps):
            ref, nxt = pair.oracle.step(tok, pos)
            pair.ctx.step(tok, pos)
            torch.cuda.synchronize()
            got = pair.ctx.logits.cpu().numpy()
            assert_logits_close(got, ref, f"{name} step {s}")
            if top2_margin(ref) > TOKEN_MARGIN:
                assert int(pair.ctx.next_token.item()) == nxt
            tok, pos = nxt, pos + 1
        assert pair.ctx.cur_len == T0 + steps == pair.oracle.cur_len
        # the appended rows: exactly rows T0 .. T0 + steps - 1 changed; codes within one step of the oracle's, scales to 5e-5
        k8b, v8b, ksb, vsb = [t.cpu().numpy() for t in pair.ctx.export_kv_int8()]
        ok8, ov8, oks, ovs = pair.oracle.export_kv_q8()
        for got_c, got_s, ref_c, ref_s, before_c, before_s in ((k8b, ksb, ok8, oks, k8, ks), (v8b, vsb, ov8, ovs, v8, vs)):
            new = slice(T0, T0 + steps)
            assert np.array_equal(np.delete(got_c, np.s_[new], axis=2), np.delete(before_c, np.s_[new], axis=2))   # nothing else written
            assert np.array_equal(np.delete(got_s, np.s_[new], axis=2), np.delete(before_s, np.s_[new], axis=2))
            diff = np.abs(got_c[:, :, new].astype(np.int32) - ref_c[:, :, new].astype(np.int32))
            assert diff.max() <= 1 and (diff != 0).mean() < 0.02, (diff.max(), (diff != 0).mean())
            assert np.abs(got_c[:, :, new]).max(axis=-1).min() == 127                                           # every row uses the whole range
            # the scale is amax / 127 of a row whose fp32 values differ between the sides by the summation error of the path
            # (fp32 against fp64 sums, growing with K and the number of layers: < 1e-5 at the 7B size); 5e-5 is 1/150 of a code step
            np.testing.assert_allclose(got_s[:, :, new], ref_s[:, :, new], rtol=5e-5)
    finally:
        pair.close()


def test_compressed_cache_differs_from_plain_cache_and_rejects_the_plain_export():
    """The format is really in use (logits differ measurably from the bf16 cache's), device-chained steps run, and the bf16
    export is refused."""
    import torch
    from paper_2604_27476_b200 import EdgefmError, Status
    cfg = CONFIGS["tiny"]
    plain = Pair(cfg, cache_len=100, max_context=110)
    comp = Pair(cfg, cache_len=100, max_context=110, kv_format="int8")
    try:
        tok = first_token(cfg)
        plain.ctx.step(tok, 100); comp.ctx.step(tok, 100)
        torch.cuda.synchronize()
        a, b = plain.ctx.logits.cpu().numpy(), comp.ctx.logits.cpu().numpy()
        assert 1e-5 < np.abs(a - b).max() < 0.2
        refs = []
        for s in range(3):                                   # free-running, tokens chained on the device
            comp.ctx.step(-1, -1)
            torch.cuda.synchronize()
            refs.append(int(comp.ctx.next_token.item()))
        t, p = int(np.argmax(b)), 101
        comp.oracle.step(tok, 100)
        for s in range(3):
            ref, nxt = comp.oracle.step(t, p)
            if top2_margin(ref) > TOKEN_MARGIN:
                assert refs[s] == nxt
            t, p = refs[s], p + 1
        with pytest.raises(EdgefmError) as ei:
            comp.ctx.export_kv()
        assert ei.value.status == Status.ERR_INVALID_ARG
        with pytest.raises(EdgefmError) as ei:
            plain.ctx.export_kv_int8()
        assert ei.value.status == Status.ERR_INVALID_ARG
    finally:
        plain.close(); comp.close()


def test_unknown_cache_format_is_rejected():
    from paper_2604_27476_b200 import EdgefmError, Status, edgefm_create
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, cache_len=0, max_context=4)
    try:
        shape = dict(n_layers=cfg.n_layers, hidden=cfg.hidden, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads, head_dim=cfg.head_dim,
                     ffn=cfg.ffn, vocab=cfg.vocab, rms_eps=cfg.rms_eps, rope_theta=cfg.rope_theta, qkv_bias=0)
        with pytest.raises(EdgefmError) as ei:
            edgefm_create(shape, pair.ptrs, 4, kv_format=7)
        assert ei.value.status == Status.ERR_INVALID_ARG
        with pytest.raises(EdgefmError) as ei:
            edgefm_create(shape, pair.ptrs, 4, kv_format="int8", reserved=[0, 1, 0, 0, 0, 0, 0])
        assert ei.value.status == Status.ERR_INVALID_ARG
    finally:
        pair.close()


def test_prefix_plus_suffix_with_compressed_cache_equals_whole_prefill():
    """edgefm_append_kv on a compressed cache compresses only the rows it appends: prefix + suffix gives the same codes,
    scales and logits as one prefill of the whole (strided views of the device arrays as sources)."""
    import torch
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, max_context=cfg.cache_len + 4, kv_format="int8")
    try:
        whole = [t.cpu().numpy() for t in pair.ctx.export_kv_int8()]
        tok, pos = first_token(cfg), cfg.first_position
        pair.ctx.step(tok, pos)
        torch.cuda.synchronize()
        logits_whole = pair.ctx.logits.cpu().numpy().copy()
        pair.ctx.prefill_kv(pair.kd[:, :, :96], pair.vd[:, :, :96])
        pair.ctx.append_kv(96, pair.kd[:, :, 96:], pair.vd[:, :, 96:])
        assert pair.ctx.cur_len == cfg.cache_len
        again = [t.cpu().numpy() for t in pair.ctx.export_kv_int8()]
        n = cfg.cache_len
        for a, b in zip(whole, again):
            assert np.array_equal(a[:, :, :n], b[:, :, :n])
        pair.ctx.step(tok, pos)
        torch.cuda.synchronize()
        assert np.array_equal(pair.ctx.logits.cpu().numpy(), logits_whole)
        ref, _ = pair.oracle.step(tok, pos)
        assert_logits_close(logits_whole, ref, "compressed prefix + suffix")
    finally:
        pair.close()
