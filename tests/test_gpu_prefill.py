"""edgefm_prefill: the prefill phase (Eq. 3 of the paper, KV <- Prefill(x_1:T); behind a prefix Eq. 5) as dense tensor-core
contractions over all prompt tokens at once.  Oracle: the same tokens stepped one by one in fp64 (causal attention makes the
two the same function).

Tolerance.  Every activation enters a contraction as two bf16 pieces (16 mantissa bits), the weights are bf16 exactly,
products accumulate in fp32 and the residual stream is fp32, so before the final rounding a cache row agrees with the oracle's
to about 1e-4 of its RMS.  The row is then rounded to bf16: where the two values straddle a rounding boundary the codes
differ by one step (2^-8 relative).  Checked per layer: relative L2 error of the appended rows <= 4e-3 (a third of the codes
one step off would give 1.6e-3) and max-abs error <= 4e-2 of the tensor's RMS (one bf16 step of a value of 5 RMS is 2e-2);
the logits of the prompt's last token, computed by the decode step on these rows, within the step's tolerances (3e-2 max-abs,
1e-2 relative L2).  Measured at the 1.5B size: rows 1.4e-3 / 2.0e-2, logits 1.9e-3 max-abs, 5.5e-4 relative L2.  (With single
bf16 activations the same case gives rows 2.1e-2 at layer 27 and logits 3.6e-2 max-abs: outside the tolerance, which is why
the contractions take two pieces.)"""
import numpy as np
import pytest

from edgefm_synth import CONFIGS
from helpers import Pair, assert_logits_close, top2_margin, TOKEN_MARGIN

pytestmark = pytest.mark.gpu

ROW_REL_L2 = 4e-3
ROW_MAX_ABS_OF_RMS = 4e-2


def bits_to_f64(b):
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def assert_rows_close(gpu_bits, ref_bits, what):
    g, r = bits_to_f64(gpu_bits), bits_to_f64(ref_bits)
    assert np.isfinite(g).all(), what
    worst = worst_mx = 0.0
    for layer in range(r.shape[0]):
        rms = float(np.sqrt(np.mean(r[layer] ** 2)))
        rel = float(np.linalg.norm(g[layer] - r[layer]) / np.linalg.norm(r[layer]))
        mx = float(np.max(np.abs(g[layer] - r[layer]))) / rms
        assert rel <= ROW_REL_L2, f"{what} layer {layer}: rel-L2 {rel}"
        assert mx <= ROW_MAX_ABS_OF_RMS, f"{what} layer {layer}: max-abs / rms {mx}"
        worst = max(worst, rel)
        worst_mx = max(worst_mx, mx)
    print(f'{what}: worst rel-L2 {worst:.2e}, worst max-abs/rms {worst_mx:.2e}')
    return worst


def run_case(cfg, T0, n, seed, follow=True):
    import torch
    pair = Pair(cfg, cache_len=T0, max_context=T0 + n + 3)
    try:
        rng = np.random.default_rng(seed)
        toks = rng.integers(0, cfg.vocab, n).tolist()
        pos0 = T0 + 7                                     # positions need not equal slots
        for i, t in enumerate(toks):
            ref_logits, ref_next = pair.oracle.step(t, pos0 + i)
        pair.ctx.prefill(toks, pos0)
        assert pair.ctx.cur_len == T0 + n == pair.oracle.cur_len
        torch.cuda.synchronize()
        pair.ctx.sync_status()
        assert pair.ctx.sync_length() == T0 + n
        kg, vg = [t.cpu().numpy().view(np.uint16) for t in pair.ctx.export_kv()]
        ko, vo = pair.oracle.export_kv()
        assert np.array_equal(kg[:, :, :T0], ko[:, :, :T0]) and np.array_equal(vg[:, :, :T0], vo[:, :, :T0])   # the prefix is untouched
        wk = assert_rows_close(kg[:, :, T0:T0 + n], ko[:, :, T0:T0 + n], "K rows")
        wv = assert_rows_close(vg[:, :, T0:T0 + n], vo[:, :, T0:T0 + n], "V rows")
        ma, rl = assert_logits_close(pair.ctx.logits.cpu().numpy(), ref_logits, "logits of the last prompt token")
        print(f"{cfg.name} T0={T0} n={n}: rows rel-L2 K {wk:.2e} V {wv:.2e}; logits max-abs {ma:.2e} rel-L2 {rl:.2e}")
        if top2_margin(ref_logits) > TOKEN_MARGIN:
            assert int(pair.ctx.next_token.item()) == ref_next
            if follow:                                    # decoding continues from the device state
                pair.ctx.step(-1, -1)
                torch.cuda.synchronize()
                ref2, _ = pair.oracle.step(ref_next, pos0 + n)
                assert_logits_close(pair.ctx.logits.cpu().numpy(), ref2, "first decode step after the prompt")
    finally:
        pair.close()


@pytest.mark.parametrize("T0,n", [(0, 2), (0, 7), (0, 8), (0, 9), (20, 200), (37, 130), (64, 1), (3, 65), (0, 128), (5, 257), (123, 384)])
def test_prompt_as_dense_contractions_tiny(T0, n):
    run_case(CONFIGS["tiny"].with_(qkv_bias=True), T0, n, 300 + n)


def test_prompt_longer_than_one_pass():
    run_case(CONFIGS["tiny"], 5, 4200, 77, follow=False)


def test_prompt_on_the_1_5b_shape():
    run_case(CONFIGS["qwen2.5-1.5b"], 32, 200, 5, follow=False)


def test_prompt_behind_a_long_prefix():
    """8200 prefix rows (the context then runs the long-context build of the step kernel for the prompt's last token): the
    queries attend to 65 key blocks, the first 64 of them wholly inside the prefix."""
    run_case(CONFIGS["tiny"].with_(qkv_bias=True), 8200, 150, 9)


@pytest.mark.parametrize("name,T0,n", [("tiny", 8200, 60), ("tiny", 1000, 128), ("qwen2.5-1.5b", 2048, 40)])
def test_short_suffix_behind_a_long_prefix(name, T0, n):
    """Sec. 3.9, Eq. 5: a request's own short suffix behind a long fixed prefix.  One query tile then faces dozens of key
    blocks: they are shared out among several CTAs per head and the partial results merged."""
    run_case(CONFIGS[name] if name != "tiny" else CONFIGS[name].with_(qkv_bias=True), T0, n, 31)


def test_prompt_on_the_0_5b_shape():
    """head_dim 64, 14 query heads on 2 kv heads, tied output layer; two query tiles and a ragged third."""
    run_case(CONFIGS["qwen2.5-0.5b"], 10, 300, 6, follow=False)


def test_prompt_on_the_7b_shape():
    """28 query heads on 4 kv heads (groups of 7), H = 3584, F = 18944 (148 column tiles)."""
    run_case(CONFIGS["qwen2.5-7b-32k"], 16, 70, 8, follow=False)


def test_prefill_argument_checks():
    from paper_2604_27476_b200 import EdgefmError, Status
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, cache_len=2, max_context=4)
    try:
        with pytest.raises(EdgefmError) as ei:
            pair.ctx.prefill([1, 2, 3], 2)
        assert ei.value.status == Status.ERR_CONTEXT_FULL and pair.ctx.cur_len == 2
        with pytest.raises(EdgefmError) as ei:
            pair.ctx.prefill([1, cfg.vocab], 2)
        assert ei.value.status == Status.ERR_INVALID_ARG
        with pytest.raises(EdgefmError) as ei:
            pair.ctx.prefill([], 2)
        assert ei.value.status == Status.ERR_INVALID_ARG
    finally:
        pair.close()



def test_prefill_then_block_verification_and_pruned_vocabulary():
    """edgefm_prefill on a context built for block verification, followed by a verified block; then on a context whose output
    layer is pruned (the logits of the prompt's last token are the subset's)."""
    import torch
    cfg = CONFIGS["tiny"].with_(qkv_bias=True)
    T0, n = 6, 90
    pair = Pair(cfg, cache_len=T0, max_context=T0 + n + 8, block_tokens=4)
    try:
        toks = np.random.default_rng(21).integers(0, cfg.vocab, n).tolist()
        for i, t in enumerate(toks):
            ref_logits, ref_next = pair.oracle.step(t, T0 + i)
        pair.ctx.prefill(toks, T0)
        torch.cuda.synchronize()
        pair.ctx.sync_status()
        assert_logits_close(pair.ctx.logits.cpu().numpy(), ref_logits, "last prompt token on a block context")
        if top2_margin(ref_logits) > TOKEN_MARGIN:
            # a block behind the prompt: the token the device holds (-1) and three arbitrary proposals
            block = [ref_next, 5, 7, 9]
            ref_rows, ref_acc, ref_nx = pair.oracle.verify_block(block, T0 + n)
            pair.ctx.verify_block([-1] + block[1:], -1)
            torch.cuda.synchronize()
            assert int(pair.ctx.n_accepted.item()) == ref_acc
            assert pair.ctx.sync_length() == T0 + n + ref_acc == pair.oracle.cur_len
            got = pair.ctx.block_logits.cpu().numpy()
            for t in range(ref_acc):
                assert_logits_close(got[t], ref_rows[t], f"block row {t} behind the prompt")
            if top2_margin(ref_rows[ref_acc - 1]) > TOKEN_MARGIN:
                assert int(pair.ctx.next_token.item()) == ref_nx
    finally:
        pair.close()
    pair = Pair(cfg, cache_len=T0, max_context=T0 + n + 2)
    try:
        ids = list(range(3, cfg.vocab, 5))
        pair.ctx.set_vocab_subset(ids)
        for i, t in enumerate(toks):
            ref_logits, _ = pair.oracle.step(t, T0 + i)
        pair.ctx.prefill(toks, T0)
        torch.cuda.synchronize()
        got = pair.ctx.logits.cpu().numpy()[:len(ids)]
        assert_logits_close(got, ref_logits[ids], "last prompt token, pruned output layer")
        assert int(pair.ctx.next_token.item()) == ids[int(np.argmax(ref_logits[ids]))] or top2_margin(ref_logits[ids]) <= TOKEN_MARGIN
    finally:
        pair.close()


@pytest.mark.parametrize("name,T0,n", [("tiny", 0, 9), ("tiny", 20, 300), ("tiny", 5, 4200), ("tiny", 3000, 50), ("qwen2.5-1.5b", 32, 200)])
def test_prompt_into_the_compressed_cache(name, T0, n):
    """The same prefill on a context with the 8-bit cache (Sec. 3.9): the new rows are compressed from their fp32 values (k
    after RoPE, v) exactly as the decode step compresses its own row, and attention reads codes x scales for every row, the
    new ones included.  Oracle: the prompt stepped token by token on the oracle's compressed cache.  The rows' fp32 values
    differ from the oracle's fp64 ones in the last bits, so a code may land on its neighbour: every code within one step,
    scales to 1e-2 relative with a mean below 5e-4 (a scale is the row's largest magnitude / 127; the rows of the dense path
    agree with the oracle's to a few 1e-4 before rounding, and a code that landed on its neighbour moves one element of an
    earlier row by 1/127 of that row's maximum, which the later layers see: measured up to 2.6e-4 on the tiny shape, 2.2e-3
    for one of 11200 rows at the 1.5B size), logits within the step's tolerances."""
    import torch
    cfg = CONFIGS[name] if name != "tiny" else CONFIGS[name].with_(qkv_bias=True)
    pair = Pair(cfg, cache_len=T0, max_context=T0 + n + 3, kv_format="int8")
    try:
        toks = np.random.default_rng(40 + n).integers(0, cfg.vocab, n).tolist()
        for i, t in enumerate(toks):
            ref_logits, ref_next = pair.oracle.step(t, T0 + 3 + i)
        pair.ctx.prefill(toks, T0 + 3)
        torch.cuda.synchronize()
        pair.ctx.sync_status()
        assert pair.ctx.sync_length() == T0 + n == pair.oracle.cur_len
        got = [t.cpu().numpy() for t in pair.ctx.export_kv_int8()]
        ref = pair.oracle.export_kv_q8()
        new = slice(T0, T0 + n)
        for g8, r8 in zip(got[:2], ref[:2]):
            assert np.array_equal(g8[:, :, :T0], r8[:, :, :T0])                       # the prefix is untouched
            diff = np.abs(g8[:, :, new].astype(np.int32) - r8[:, :, new].astype(np.int32))
            assert diff.max() <= 1 and (diff != 0).mean() < 0.08, (diff.max(), (diff != 0).mean())
        for gs, rs in zip(got[2:], ref[2:]):
            rel = np.abs(gs[:, :, new] - rs[:, :, new]) / np.maximum(rs[:, :, new], 1e-30)
            assert rel.max() <= 1e-2 and rel.mean() <= 5e-4, (rel.max(), rel.mean())
            worst_scale = max(locals().get('worst_scale', 0.0), float(rel.max()))
        ma, rl = assert_logits_close(pair.ctx.logits.cpu().numpy(), ref_logits, "last prompt token, compressed cache")
        print(f"{name} int8 T0={T0} n={n}: logits max-abs {ma:.2e} rel-L2 {rl:.2e}; scales worst rel {worst_scale:.2e}")
        if top2_margin(ref_logits) > TOKEN_MARGIN:
            assert int(pair.ctx.next_token.item()) == ref_next
    finally:
        pair.close()
