"""Parity of the CUDA decode step (through the C ABI) against the CPU oracle, element by element."""
import numpy as np
import pytest

from edgefm_synth import CONFIGS, first_token, make_kv, make_weights
from helpers import (LOGIT_MAX_ABS, Pair, TOKEN_MARGIN, assert_appended_rows_close, assert_logits_close, top2_margin)

pytestmark = pytest.mark.gpu

TINY = CONFIGS["tiny"]


def run_teacher_forced(pair: Pair, steps: int, first_tok: int, first_pos: int):
    """Oracle free-runs greedily; the CUDA path is fed the oracle's tokens.  Returns per-step stats."""
    import torch
    tok, pos = first_tok, first_pos
    stats = []
    for s in range(steps):
        ref_logits, ref_next = pair.oracle.step(tok, pos)
        pair.ctx.step(tok, pos)
        torch.cuda.synchronize()
        gpu_logits = pair.ctx.logits.cpu().numpy()
        gpu_next = int(pair.ctx.next_token.item())
        ma, rl = assert_logits_close(gpu_logits, ref_logits, f"step {s}")
        margin = top2_margin(ref_logits)
        if margin > TOKEN_MARGIN:
            assert gpu_next == ref_next, f"step {s}: token {gpu_next} != {ref_next} at margin {margin}"
        assert gpu_next == int(np.argmax(gpu_logits)), "next token is not the first argmax of the GPU's own logits"
        stats.append((ma, rl, margin, gpu_next == ref_next))
        tok, pos = ref_next, pos + 1
    return stats


def check_cache_against_oracle(pair: Pair, first_slot: int, n_new: int):
    import torch
    kg, vg = pair.ctx.export_kv()
    torch.cuda.synchronize()
    kg = kg.cpu().numpy().view(np.uint16)
    vg = vg.cpu().numpy().view(np.uint16)
    ko, vo = pair.oracle.export_kv()
    assert np.array_equal(kg[:, :, :first_slot], ko[:, :, :first_slot])       # the prefix is untouched
    assert np.array_equal(vg[:, :, :first_slot], vo[:, :, :first_slot])
    new = slice(first_slot, first_slot + n_new)
    assert_appended_rows_close(kg[:, :, new], ko[:, :, new])
    assert_appended_rows_close(vg[:, :, new], vo[:, :, new])


def test_tiny_single_step_matches_oracle():
    pair = Pair(TINY)
    try:
        stats = run_teacher_forced(pair, 1, first_token(TINY), TINY.first_position)
        assert pair.ctx.cur_len == pair.oracle.cur_len == TINY.cache_len + 1
        check_cache_against_oracle(pair, TINY.cache_len, 1)
        assert stats[0][0] < 1e-3                                  # far inside the tolerance on this small model
    finally:
        pair.close()


def test_kv_write_set_is_exactly_the_new_slot():
    """Unfilled slots carry a NaN sentinel; after one step exactly row cur_len of every (layer, kv head)
    of K and of V has changed, and nothing else (bit-exact write indices)."""
    import torch
    cfg = TINY
    T0, Tmax = 37, 64
    pair = Pair(cfg, cache_len=T0, max_context=Tmax)
    try:
        sentinel = torch.full((cfg.n_layers, cfg.n_kv_heads, Tmax, cfg.head_dim), 0x7FC1, dtype=torch.int16, device="cuda")
        sentinel[:, :, :T0] = pair.kd
        pair.ctx.prefill_kv(sentinel, sentinel)      # fills every slot, sentinel behind the prefix
        pair.ctx.prefill_kv(pair.kd, pair.vd)        # cache length back to T0, rows >= T0 keep the sentinel
        k0, v0 = [t.cpu().numpy().view(np.uint16) for t in pair.ctx.export_kv()]
        guard = torch.full((cfg.vocab + 64,), 12345.0, device="cuda")
        from paper_2604_27476_b200 import edgefm_decode_step
        edgefm_decode_step(pair.ctx.handle, 5, T0, torch.cuda.current_stream().cuda_stream, guard.data_ptr(), None)
        torch.cuda.synchronize()
        assert torch.all(guard[cfg.vocab:] == 12345.0)                       # nothing written past the logits
        k1, v1 = [t.cpu().numpy().view(np.uint16) for t in pair.ctx.export_kv()]
        for a0, a1 in ((k0, k1), (v0, v1)):
            changed = np.argwhere(a0 != a1)
            assert set(changed[:, 2].tolist()) == {T0}
            assert len(changed) == cfg.n_layers * cfg.n_kv_heads * cfg.head_dim   # every element of the row was a sentinel
            assert not np.any(a1[:, :, T0] == 0x7FC1)
        assert pair.ctx.cur_len == T0 + 1
    finally:
        pair.close()


VARIANTS = {
    "bias": dict(qkv_bias=True),
    "tied": dict(tied=True),
    "mha_g1": dict(n_q_heads=2, n_kv_heads=2),
    "g3_d128": dict(n_q_heads=6, n_kv_heads=2, head_dim=128, hidden=264),
    "g8": dict(n_q_heads=8, n_kv_heads=1, hidden=200, ffn=72, vocab=1000),
    "g7_odd": dict(n_q_heads=7, n_kv_heads=1, hidden=136, ffn=8, vocab=33, n_layers=3, qkv_bias=True),
    # long rows (K slices per work item) and enough tiles per warp to wrap the shared-memory ring many times
    "ring_wrap_ksplit": dict(hidden=512, ffn=6144, vocab=50000, n_layers=3, qkv_bias=True),
    "g5_kv3": dict(n_q_heads=15, n_kv_heads=3, head_dim=128, hidden=512, ffn=1000, vocab=777),
}


@pytest.mark.parametrize("name", sorted(VARIANTS))
def test_tiny_variants_multi_step_from_short_cache(name):
    cfg = TINY.with_(**VARIANTS[name])
    pair = Pair(cfg, seed=100 + len(name), cache_len=5, max_context=80)
    try:
        run_teacher_forced(pair, 70, 3 % cfg.vocab, 11)   # crosses a 64-position chunk boundary
        check_cache_against_oracle(pair, 5, 70)
    finally:
        pair.close()


def test_empty_cache_first_step_and_position_independent_of_slot():
    pair = Pair(TINY, cache_len=0, max_context=8)
    try:
        run_teacher_forced(pair, 8, 7, 1000)              # slot 0.., positions 1000..
        check_cache_against_oracle(pair, 0, 8)
    finally:
        pair.close()


@pytest.mark.parametrize("cache_len", [31, 32, 33, 63, 64, 65, 127, 129, 500, 1023])
def test_attention_chunk_boundaries(cache_len):
    cfg = TINY.with_(n_layers=1, vocab=256)
    pair = Pair(cfg, seed=cache_len, cache_len=cache_len, max_context=1100)
    try:
        run_teacher_forced(pair, 2, 9, cache_len)
    finally:
        pair.close()


def test_free_run_matches_teacher_forced_and_device_chaining():
    """token = -1 / position = -1 chain the previous step's result on the device."""
    import torch
    cfg = TINY
    pair = Pair(cfg, max_context=cfg.cache_len + 20)
    try:
        tok, pos = first_token(cfg), cfg.first_position
        toks_ref, margins = [], []
        o_tok = tok
        for s in range(20):
            lg, nx = pair.oracle.step(o_tok, pos + s)
            toks_ref.append(nx); margins.append(top2_margin(lg)); o_tok = nx
        out = torch.zeros(20, dtype=torch.int32, device="cuda")
        from paper_2604_27476_b200 import edgefm_decode_step
        st = torch.cuda.current_stream().cuda_stream
        edgefm_decode_step(pair.ctx.handle, tok, pos, st, None, out.data_ptr())
        for s in range(1, 20):                              # no host sync, no logits
            edgefm_decode_step(pair.ctx.handle, -1, -1, st, None, out.data_ptr() + 4 * s)
        torch.cuda.synchronize()
        got = out.cpu().tolist()
        for s in range(20):
            if got[s] != toks_ref[s]:
                assert margins[s] <= TOKEN_MARGIN, f"diverged at step {s} with margin {margins[s]}"
                break
        assert pair.ctx.cur_len == cfg.cache_len + 20
    finally:
        pair.close()


def test_run_twice_is_bit_identical():
    import torch
    outs = []
    for _ in range(2):
        pair = Pair(TINY.with_(qkv_bias=True), cache_len=300, max_context=320)
        try:
            acc = []
            for s in range(6):
                pair.ctx.step(17 + s, 300 + s)
                torch.cuda.synchronize()
                acc.append(pair.ctx.logits.cpu().numpy().copy())
            outs.append(np.stack(acc))
        finally:
            pair.close()
    assert np.array_equal(outs[0].view(np.uint32), outs[1].view(np.uint32))


def test_statefulness_export_then_prefill():
    import torch
    cfg = TINY
    pair = Pair(cfg, cache_len=40, max_context=64)
    try:
        for s in range(3):
            pair.ctx.step(100 + s, 40 + s)
        k, v = pair.ctx.export_kv()
        pair.ctx.step(200, 43)
        torch.cuda.synchronize()
        a = pair.ctx.logits.cpu().numpy().copy()
        from paper_2604_27476_b200 import DecodeContext
        ctx2 = DecodeContext(cfg, pair.ptrs, 64)
        ctx2.prefill_kv(k[:, :, :43], v[:, :, :43])          # strided view: stride_pos = d, stride_head = 64*d
        ctx2.step(200, -1)                                    # position -1 after prefill = cache length = 43
        torch.cuda.synchronize()
        b = ctx2.logits.cpu().numpy()
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
        ctx2.close()
    finally:
        pair.close()


@pytest.mark.parametrize("variant", ["g2_d64", "g7_d128_bias"])
def test_long_context_build_crosses_the_attention_mode_switch(variant):
    """max_context > 8192 selects the long-context build of the kernel (8 warps per CTA, both attention modes).
    Starting at 8188 cached positions, the steps cross the switch from one-head-per-CTA attention (merged in the
    O-projection prologue) to grouped attention (merged by the last CTA of a group)."""
    cfg = TINY if variant == "g2_d64" else TINY.with_(n_q_heads=7, n_kv_heads=1, head_dim=128, hidden=320, ffn=512, vocab=3000,
                                                         qkv_bias=True)
    pair = Pair(cfg, seed=77, cache_len=8188, max_context=8200)
    try:
        run_teacher_forced(pair, 9, 5, 8188)          # attends 8189 .. 8197 positions
        check_cache_against_oracle(pair, 8188, 9)
    finally:
        pair.close()
