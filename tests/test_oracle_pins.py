"""Pins of the CPU oracle against closed forms, invariants and brute force (no GPU).

Each test is chosen so that a plausible mistake in the oracle -- a dropped term, a wrong sign or
index, a transposed operand, a wrong rounding point -- fails it.
"""
import math
from pathlib import Path

import numpy as np
import pytest

from edgefm_synth import CONFIGS, bf16_to_f32, make_weights, normal_bf16
from oracle import OracleModel, binding as O, tiny_ref

GOLDEN = Path(__file__).parent / "golden"


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Independent fp32 -> bf16 RNE in numpy integer arithmetic."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32).astype(np.uint64)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def rand_bf16(rng, shape, std=1.0):
    return to_bf16_bits(rng.normal(0, std, shape).astype(np.float32))


# ---- bf16 rounding --------------------------------------------------------------------------
def test_bf16_round_to_nearest_even_cases():
    assert O.bf16_to_f32(O.f32_to_bf16(1.0 + 2.0 ** -8)) == 1.0              # tie -> even (down)
    assert O.bf16_to_f32(O.f32_to_bf16(1.0 + 3 * 2.0 ** -8)) == 1.015625     # tie -> even (up)
    assert O.bf16_to_f32(O.f32_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -20)) == 1.0078125  # above tie -> up
    assert O.f32_to_bf16(0.0) == 0x0000 and O.f32_to_bf16(-0.0) == 0x8000
    assert O.f32_to_bf16(float("inf")) == 0x7F80 and O.f32_to_bf16(float("-inf")) == 0xFF80
    assert math.isnan(O.bf16_to_f32(O.f32_to_bf16(float("nan"))))
    assert O.f32_to_bf16(3.3895314e38) == 0x7F7F                              # largest finite bf16 stays finite


def test_bf16_roundtrip_every_pattern():
    for b in range(0, 1 << 16):
        f = O.bf16_to_f32(b)
        if math.isnan(f):
            continue
        assert O.f32_to_bf16(f) == b


# ---- GEMV -----------------------------------------------------------------------------------
@pytest.mark.parametrize("rows,cols", [(1, 1), (3, 5), (7, 8), (17, 33), (64, 100)])
def test_gemv_vs_naive_triple_loop(rows, cols):
    rng = np.random.default_rng(rows * 100 + cols)
    W = rand_bf16(rng, (rows, cols))
    b = rand_bf16(rng, (rows,))
    x = rng.normal(size=cols).astype(np.float32)
    Wf = bf16_to_f32(W)
    for bias in (None, b):
        y = O.gemv(W, x, bias)
        for r in range(rows):                      # plain python loops, exact rational-free fp64 sum
            acc = 0.0
            for k in range(cols):
                acc += float(Wf[r, k]) * float(x[k])
            if bias is not None:
                acc += float(bf16_to_f32(b[r:r + 1])[0])
            assert y[r] == np.float32(acc)


def test_gemv_not_transposed_identity_zero():
    rng = np.random.default_rng(1)
    n = 9
    x = rng.normal(size=n).astype(np.float32)
    eye = to_bf16_bits(np.eye(n, dtype=np.float32))
    assert np.array_equal(O.gemv(eye, x), x)
    b = rand_bf16(rng, (n,))
    assert np.array_equal(O.gemv(np.zeros((n, n), np.uint16), x, b), bf16_to_f32(b))
    # a single 1 at W[2][5] must pick x[5] into y[2] (a transposed read would pick x[2] into y[5])
    W = np.zeros((n, n), np.float32); W[2, 5] = 1.0
    y = O.gemv(to_bf16_bits(W), x)
    assert y[2] == x[5] and np.count_nonzero(y) == 1


# ---- RMSNorm --------------------------------------------------------------------------------
@pytest.mark.parametrize("c", [0.5, -3.0, 1e-3, 100.0])
def test_rmsnorm_constant_vector_closed_form(c):
    n, eps = 256, 1e-6
    ones = np.full(n, 0x3F80, np.uint16)
    out = O.rmsnorm(np.full(n, c, np.float32), ones, eps)
    c32 = float(np.float32(c))
    expect = np.float32(c32 / math.sqrt(c32 * c32 + eps))      # eps inside the root, mean not sum
    assert np.all(out == expect)


def test_rmsnorm_weight_applied_after_and_unit_rms():
    rng = np.random.default_rng(2)
    n, eps = 96, 1e-6
    x = rng.normal(size=n).astype(np.float32)
    ones = np.full(n, 0x3F80, np.uint16)
    base = O.rmsnorm(x, ones, eps)
    assert abs(float(np.sqrt(np.mean(base.astype(np.float64) ** 2))) - 1.0) < 1e-5
    w = rand_bf16(rng, (n,))
    out = O.rmsnorm(x, w, eps)
    np.testing.assert_allclose(out, base.astype(np.float64) * bf16_to_f32(w), rtol=2e-7)   # no "+1" on w
    np.testing.assert_allclose(O.rmsnorm(7.0 * x, ones, eps), base, rtol=1e-5)              # scale invariance


# ---- RoPE -----------------------------------------------------------------------------------
def test_rope_printed_example_d4():
    lines = [l for l in (GOLDEN / "rope_d4_theta1e4_pos1.txt").read_text().splitlines() if l and l[0] != "#"]
    expect = np.array([float(l) for l in lines])
    got = O.rope(np.array([1, 2, 3, 4], np.float32), 1, 10000.0)
    np.testing.assert_allclose(got, expect, rtol=0, atol=3e-7)


def test_rope_identity_norm_composition_relative():
    rng = np.random.default_rng(3)
    d, theta = 64, 1e6
    q = rng.normal(size=d).astype(np.float32)
    k = rng.normal(size=d).astype(np.float32)
    assert np.array_equal(O.rope(q, 0, theta), q)                                     # pos 0 = identity
    r = O.rope(q, 1234, theta)
    np.testing.assert_allclose(r[: d // 2] ** 2 + r[d // 2:] ** 2, q[: d // 2] ** 2 + q[d // 2:] ** 2, rtol=1e-5)
    np.testing.assert_allclose(O.rope(O.rope(q, 700, theta), 55, theta), O.rope(q, 755, theta), atol=2e-6)
    a = float(np.dot(O.rope(q, 1000, theta).astype(np.float64), O.rope(k, 990, theta)))
    b = float(np.dot(O.rope(q, 33010, theta).astype(np.float64), O.rope(k, 33000, theta)))
    assert abs(a - b) < 1e-4                                                          # depends on m - n only


def test_rope_frequency_ladder_and_direction():
    # unit vector on pair i comes back as (cos, sin) of pos * theta^(-2i/d): pins frequency index,
    # pairing (i, i + d/2) and the rotation direction.
    d, theta, pos = 8, 100.0, 3
    for i in range(d // 2):
        u = np.zeros(d, np.float32); u[i] = 1.0
        r = O.rope(u, pos, theta)
        phi = pos * theta ** (-2.0 * i / d)
        expect = np.zeros(d); expect[i] = math.cos(phi); expect[i + d // 2] = math.sin(phi)
        np.testing.assert_allclose(r, expect, atol=1e-7)


def test_rope_large_position_accuracy():
    # at position 32832 the fastest pair has turned ~5225 times; fp64 angle keeps full accuracy
    d, theta, pos = 128, 1e6, 32832
    u = np.zeros(d, np.float32); u[0] = 1.0
    r = O.rope(u, pos, theta)
    from fractions import Fraction
    # reduce pos mod 2*pi with extended precision (pi to 40 digits as a rational)
    pi = Fraction(3141592653589793238462643383279502884197, 10 ** 39)
    red = Fraction(pos) - (Fraction(pos) // (2 * pi)) * 2 * pi
    assert abs(r[0] - math.cos(float(red))) < 1e-7 and abs(r[d // 2] - math.sin(float(red))) < 1e-7


# ---- softmax / SiLU / argmax ----------------------------------------------------------------
def test_softmax_rows_sum_to_one_shift_uniform():
    rng = np.random.default_rng(4)
    s = (rng.normal(size=1000) * 5).astype(np.float32)
    p = O.softmax(s)
    assert abs(float(p.astype(np.float64).sum()) - 1.0) < 1e-6
    np.testing.assert_allclose(O.softmax(s + np.float32(8.0)), p, rtol=1e-5)
    assert np.all(O.softmax(np.full(10, 3.25, np.float32)) == np.float32(0.1))
    p2 = O.softmax(np.array([0.0, math.log(3.0)], np.float32))
    np.testing.assert_allclose(p2, [0.25, 0.75], rtol=1e-6)
    assert np.isfinite(O.softmax(np.array([1000.0, 999.0], np.float32))).all()


def test_silu_closed_forms():
    assert O.silu(0.0) == 0.0
    assert abs(O.silu(1.0) - 0.7310585786300049) < 1e-15
    assert abs(O.silu(-2.0) - (-2.0 / (1.0 + math.exp(2.0)))) < 1e-15
    assert abs(O.silu(40.0) - 40.0) < 1e-12
    assert O.silu(-800.0) == 0.0 or abs(O.silu(-800.0)) < 1e-300       # no overflow / NaN
    assert O.silu(800.0) == 800.0


def test_argmax_planted_and_ties():
    n = 4096
    base = np.full(n, -1.0, np.float32)
    for idx in (0, 1, 255, 256, 257, n - 1):
        v = base.copy(); v[idx] = 2.0
        assert O.argmax(v) == idx
    v = base.copy(); v[100] = 5.0; v[3000] = 5.0
    assert O.argmax(v) == 100                                           # lowest index wins
    v = base.copy(); v[7] = float("nan"); v[9] = 0.0
    assert O.argmax(v) == 9                                             # NaN never wins
    assert O.argmax(np.full(5, -np.inf, np.float32)) == 0


def test_restricted_greedy_against_brute_force():
    """Vocabulary pruning (caption of Fig. 2): the greedy choice over a subset of ids.  Pinned by the full vocabulary
    reducing to the plain argmax, a planted maximum outside the subset being ignored, ties, and a brute-force loop."""
    rng = np.random.default_rng(5)
    V = 5000
    logits = rng.standard_normal(V).astype(np.float32)
    sub, nxt = O.restricted_greedy(logits, np.arange(V))
    assert np.array_equal(sub, logits) and nxt == O.argmax(logits) == int(np.argmax(logits))
    ids = np.sort(rng.choice(V, 700, replace=False))
    outside = int(np.setdiff1d(np.arange(V), ids)[17])
    planted = logits.copy(); planted[outside] = 100.0                   # the global maximum is not in the subset
    sub, nxt = O.restricted_greedy(planted, ids)
    best, best_id = -np.inf, -1
    for t in ids:                                                       # brute force
        if planted[t] > best:
            best, best_id = planted[t], int(t)
    assert nxt == best_id and nxt != outside
    assert np.array_equal(sub, np.array([planted[t] for t in ids], np.float32))
    tie = logits.copy(); tie[ids[600]] = 50.0; tie[ids[40]] = 50.0
    assert O.restricted_greedy(tie, ids)[1] == int(ids[40])             # equal maxima: the lowest id
    assert O.restricted_greedy(logits, [1234])[1] == 1234               # a single candidate always wins


# ---- attention ------------------------------------------------------------------------------
def test_attention_single_position_returns_v_exactly():
    rng = np.random.default_rng(5)
    nq, nkv, d = 4, 2, 16
    q = rng.normal(size=(nq, d)).astype(np.float32)
    K = rand_bf16(rng, (nkv, 1, d)); V = rand_bf16(rng, (nkv, 1, d))
    out = O.attention(q, K, V)
    Vf = bf16_to_f32(V)
    for h in range(nq):
        assert np.array_equal(out[h], Vf[h // 2, 0])                    # contiguous GQA groups


def test_attention_zero_query_is_mean_and_groups_share_kv():
    rng = np.random.default_rng(6)
    nq, nkv, d, n = 6, 2, 8, 37
    K = rand_bf16(rng, (nkv, n, d)); V = rand_bf16(rng, (nkv, n, d))
    out = O.attention(np.zeros((nq, d), np.float32), K, V)
    Vm = bf16_to_f32(V).astype(np.float64).mean(axis=1)
    for h in range(nq):
        np.testing.assert_allclose(out[h], Vm[h // 3], rtol=1e-6, atol=1e-7)
    q1 = rng.normal(size=d).astype(np.float32)
    out = O.attention(np.tile(q1, (nq, 1)), K, V)
    assert np.array_equal(out[0], out[1]) and np.array_equal(out[1], out[2])       # same group, same q
    assert not np.array_equal(out[2], out[3])                                       # next group differs


def test_attention_vs_numpy_definition_and_scale():
    rng = np.random.default_rng(7)
    nq, nkv, d, n = 4, 4, 32, 50                                                    # n_q = n_kv: plain MHA
    q = rng.normal(size=(nq, d)).astype(np.float32)
    K = rand_bf16(rng, (nkv, n, d)); V = rand_bf16(rng, (nkv, n, d))
    out = O.attention(q, K, V)
    Kf, Vf = bf16_to_f32(K).astype(np.float64), bf16_to_f32(V).astype(np.float64)
    s = np.einsum("hd,htd->ht", q.astype(np.float64), Kf) / math.sqrt(d)
    p = np.exp(s - s.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
    np.testing.assert_allclose(out, np.einsum("ht,htd->hd", p, Vf), rtol=2e-6, atol=2e-7)
    # two keys, scores differ by exactly ln(3) after the 1/sqrt(d) scale -> weights 1/4, 3/4
    d = 16
    q = np.zeros((1, d), np.float32); q[0, 0] = 4.0                                 # q.k / sqrt(16) = k0
    K = np.zeros((1, 2, d), np.float32); K[0, 1, 0] = 1.0
    V = np.zeros((1, 2, d), np.float32); V[0, 0, 0] = 1.0; V[0, 1, 1] = 1.0
    out = O.attention(q, to_bf16_bits(K), to_bf16_bits(V))
    e = math.e
    np.testing.assert_allclose(out[0, :2], [1 / (1 + e), e / (1 + e)], rtol=1e-6)


# ---- whole step -----------------------------------------------------------------------------
TINY = CONFIGS["tiny"]


@pytest.fixture(scope="module")
def tiny_weights():
    return make_weights(TINY)


def test_step_reduces_to_lm_head_when_projections_are_zero(tiny_weights):
    # Wo = Wd = 0 in every layer => logits = W_lm . RMSNorm(E[token]); isolates embed, final norm,
    # lm_head orientation and argmax.
    w = {**tiny_weights, "layers": [dict(l, wo=np.zeros_like(l["wo"]), w_down=np.zeros_like(l["w_down"]))
                                     for l in tiny_weights["layers"]]}
    m = OracleModel(TINY, w, 8)
    tok = 1234
    logits, nxt = m.step(tok, 0)
    e = bf16_to_f32(w["embed"][tok]).astype(np.float64)
    xf = (e / math.sqrt(float(np.mean(e * e)) + TINY.rms_eps)).astype(np.float32).astype(np.float64)
    expect = bf16_to_f32(w["lm_head"]).astype(np.float64) @ xf
    np.testing.assert_allclose(logits, expect, rtol=1e-6, atol=1e-7)
    assert nxt == int(np.argmax(expect))


@pytest.mark.parametrize("variant", ["plain", "bias", "tied", "mha_d32"])
def test_cached_decoding_equals_full_causal_recompute(variant):
    cfg = TINY
    if variant == "bias":
        cfg = cfg.with_(qkv_bias=True)
    elif variant == "tied":
        cfg = cfg.with_(tied=True)
    elif variant == "mha_d32":
        cfg = cfg.with_(n_q_heads=4, n_kv_heads=4, head_dim=32, hidden=192, ffn=200, vocab=517, n_layers=3)
    w = make_weights(cfg, seed=11)
    rng = np.random.default_rng(12)
    T = 14
    toks = rng.integers(0, cfg.vocab, T).tolist()
    pos = (np.arange(T) + 40).tolist() if variant != "plain" else np.arange(T).tolist()
    m = OracleModel(cfg, w, T)
    got = np.stack([m.step(t, p)[0] for t, p in zip(toks, pos)])
    ref = tiny_ref.full_forward(cfg, w, toks, pos)
    assert np.abs(got - ref).max() < 1e-5
    assert m.cur_len == T


# ---- compressed cache (Sec. 3.9: KV~ = C(KV), reconstruction on demand) ---------------------------------------
def test_int8_row_compression_worked_example_and_properties():
    # by hand: amax = 2, 127 / 2 = 63.5;  1 -> 63.5 -> 64 (tie to even), -2 -> -127, 0.5 -> 31.75 -> 32, 0 -> 0;  scale = 2 / 127
    codes, scale = O.quantize_row(np.array([1.0, -2.0, 0.5, 0.0], np.float32))
    assert codes.tolist() == [64, -127, 32, 0]
    assert scale == np.float32(2.0) / np.float32(127.0)
    codes, scale = O.quantize_row(np.zeros(8, np.float32))
    assert codes.tolist() == [0] * 8 and scale == 0.0
    rng = np.random.default_rng(5)
    for d in (4, 64, 128):
        x = rng.standard_normal(d).astype(np.float32) * np.float32(rng.uniform(1e-3, 50))
        codes, scale = O.quantize_row(x)
        assert np.abs(codes).max() == 127 and np.abs(codes[np.argmax(np.abs(x))]) == 127      # the largest value takes the end of the range
        assert np.abs(codes.astype(np.float64) * scale - x).max() <= scale * 0.5 * (1 + 1e-6)   # nearest code
        c2, s2 = O.quantize_row(-x)
        assert (c2 == -codes).all() and s2 == scale                                              # odd symmetry
        c3, s3 = O.quantize_row(x * np.float32(4))                                               # a power of two moves the scale only
        assert (c3 == codes).all() and s3 == scale * np.float32(4)


def test_attention_over_compressed_cache_reduces_to_plain_attention_on_exact_rows():
    # rows of integers with amax 127, times a power of two, compress without loss (codes = integers, scale = the power of
    # two) and are exact in bf16 as well: both attention routines must then see the same numbers
    rng = np.random.default_rng(6)
    n_q, n_kv, d, n = 4, 2, 32, 9
    Ki = rng.integers(-127, 128, (n_kv, n, d)); Vi = rng.integers(-127, 128, (n_kv, n, d))
    Ki[..., 0] = 127; Vi[..., 1] = -127                                    # every row reaches the end of the range
    sk = 2.0 ** rng.integers(-6, 0, (n_kv, n)); sv = 2.0 ** rng.integers(-4, 2, (n_kv, n))
    K = (Ki * sk[..., None]).astype(np.float32); V = (Vi * sv[..., None]).astype(np.float32)
    q = rng.standard_normal((n_q, d)).astype(np.float32)
    K8 = np.empty_like(Ki, dtype=np.int8); V8 = np.empty_like(Vi, dtype=np.int8)
    Ks = np.empty((n_kv, n), np.float32); Vs = np.empty((n_kv, n), np.float32)
    for g in range(n_kv):
        for t in range(n):
            K8[g, t], Ks[g, t] = O.quantize_row(K[g, t])
            V8[g, t], Vs[g, t] = O.quantize_row(V[g, t])
    assert (K8 == Ki).all() and (V8 == Vi).all() and (Ks == sk).all() and (Vs == sv).all()
    to_bits = lambda a: (a.view(np.uint32) >> 16).astype(np.uint16)
    assert ((to_bits(K).astype(np.uint32) << 16).view(np.float32) == K).all()           # exact in bf16
    plain = O.attention(q, to_bits(K), to_bits(V))
    comp = O.attention_q8(q, K8, Ks, V8, Vs)
    assert np.array_equal(plain, comp)


@pytest.mark.parametrize("variant", ["plain", "bias_gqa"])
def test_cached_decoding_with_compressed_cache_equals_full_causal_recompute(variant):
    cfg = TINY if variant == "plain" else TINY.with_(qkv_bias=True, n_layers=3)
    w = make_weights(cfg, seed=13)
    rng = np.random.default_rng(14)
    T = 12
    toks = rng.integers(0, cfg.vocab, T).tolist()
    pos = (np.arange(T) + 7).tolist()
    m = OracleModel(cfg, w, T, kv_format="int8")
    got = np.stack([m.step(t, p)[0] for t, p in zip(toks, pos)])
    ref = tiny_ref.full_forward(cfg, w, toks, pos, kv_int8=True)
    assert np.abs(got - ref).max() < 1e-5
    # and the compression is visible: the same run over the bf16 cache differs by far more than that
    plain = tiny_ref.full_forward(cfg, w, toks, pos)
    assert np.abs(plain - ref).max() > 1e-4
    k8, v8, ks, vs = m.export_kv_q8()
    assert np.abs(k8[:, :, :T]).max(axis=-1).min() == 127 and (ks[:, :, :T] > 0).all()


def test_compressed_cache_load_compresses_the_given_rows(tiny_weights):
    from edgefm_synth import make_kv
    cfg, w = TINY, tiny_weights
    k, v = make_kv(cfg, n_positions=5)
    m = OracleModel(cfg, w, 8, kv_format="int8")
    m.load_kv(k, v)
    k8, v8, ks, vs = m.export_kv_q8()
    for (l, g, t) in [(0, 0, 0), (1, 1, 4), (0, 1, 2)]:
        row = (k[l, g, t].astype(np.uint32) << 16).view(np.float32)
        codes, scale = O.quantize_row(row)
        assert (k8[l, g, t] == codes).all() and ks[l, g, t] == scale
    assert (k8[:, :, 5:] == 0).all() and (vs[:, :, 5:] == 0).all() and m.cur_len == 5


def test_block_verification_is_what_plain_steps_would_have_produced(tiny_weights):
    """Sec. 3.11: verify token by token, stop at the first rejection, commit the accepted prefix.  Whatever the proposals,
    the cache and the next token after a block equal those of n_accepted plain greedy steps."""
    cfg, w = TINY, tiny_weights
    plain = OracleModel(cfg, w, 16)
    seq, tok = [], 17
    for p in range(6):                       # the greedy continuation 17 -> seq[0] -> seq[1] ...
        _, tok = plain.step(tok if p else 17, p)
        seq.append(tok)
    m = OracleModel(cfg, w, 16)
    logits, n_acc, nxt = m.verify_block([17, seq[0], seq[1]], 0)            # all proposals right
    assert (n_acc, nxt, m.cur_len, logits.shape) == (3, seq[2], 3, (3, cfg.vocab))
    logits, n_acc, nxt = m.verify_block([seq[2], (seq[3] + 1) % cfg.vocab, seq[4]], 3)   # first proposal wrong: the right one behind it is not looked at
    assert (n_acc, nxt, m.cur_len) == (1, seq[3], 4)
    logits, n_acc, nxt = m.verify_block([seq[3], seq[4], (seq[5] + 1) % cfg.vocab], 4)   # second proposal wrong
    assert (n_acc, nxt, m.cur_len) == (2, seq[5], 6)
    ka, va = m.export_kv(); kb, vb = plain.export_kv()
    assert np.array_equal(ka[:, :, :6], kb[:, :, :6]) and np.array_equal(va[:, :, :6], vb[:, :, :6])
    with pytest.raises(ValueError):
        m.truncate(7)


def test_position_is_independent_of_slot(tiny_weights):
    # Same cache content, same token, different RoPE position => different logits; the slot written
    # is cur_len in both cases (vision-token prefixes make position != slot).
    rng = np.random.default_rng(13)
    outs = []
    for pos in (3, 50):
        m = OracleModel(TINY, tiny_weights, 8)
        for t in (5, 6, 7):
            m.step(t, 0)
        before = m.export_kv()
        lg, _ = m.step(99, pos)
        after = m.export_kv()
        outs.append(lg)
        changed = np.argwhere((before[0] != after[0]).any(axis=-1))
        assert set(changed[:, 2].tolist()) == {3}                        # only slot 3, every layer/head
        assert len(changed) == TINY.n_layers * TINY.n_kv_heads
    assert np.abs(outs[0] - outs[1]).max() > 1e-3


def test_statefulness_export_reload(tiny_weights):
    m = OracleModel(TINY, tiny_weights, 16)
    for i, t in enumerate((11, 22, 33, 44)):
        m.step(t, i)
    k, v = m.export_kv()
    lg_a, nx_a = m.step(55, 4)
    m2 = OracleModel(TINY, tiny_weights, 16)
    m2.load_kv(k[:, :, :4], v[:, :, :4])
    lg_b, nx_b = m2.step(55, 4)
    assert np.array_equal(lg_a, lg_b) and nx_a == nx_b


def test_appended_kv_is_bf16_of_rotated_k_and_plain_v(tiny_weights):
    # first step on an empty cache: attention over one position returns bf16(v) exactly, and the
    # stored K row is bf16(RoPE(k)).
    cfg = TINY
    m = OracleModel(cfg, tiny_weights, 4)
    tok, pos = 77, 9
    m.step(tok, pos)
    k, v = m.export_kv()
    lw = tiny_weights["layers"][0]
    x = bf16_to_f32(tiny_weights["embed"][tok])
    xn = O.rmsnorm(x, lw["input_norm"], cfg.rms_eps)
    qkv = O.gemv(lw["wqkv"], xn)
    nq, nkv, d = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    for g in range(nkv):
        kk = O.rope(qkv[(nq + g) * d:(nq + g + 1) * d], pos, cfg.rope_theta)
        assert np.array_equal(k[0, g, 0], to_bf16_bits(kk))
        assert np.array_equal(v[0, g, 0], to_bf16_bits(qkv[(nq + nkv + g) * d:(nq + nkv + g + 1) * d]))


def test_full_cache_is_rejected(tiny_weights):
    m = OracleModel(TINY, tiny_weights, 1)
    m.step(1, 0)
    with pytest.raises(RuntimeError):
        m.step(2, 1)


# ---- the generator (statistical sanity; it is an input recipe, not part of the method) --------
def test_generator_is_counter_based_and_normal():
    a = normal_bf16(5, 17, (100000,), 0.02)
    b = normal_bf16(5, 17, (1000,), 0.02, offset=5000)
    assert np.array_equal(a[5000:6000], b)
    f = bf16_to_f32(a).astype(np.float64)
    assert abs(f.mean()) < 3e-4 and abs(f.std() - 0.02) < 3e-4
    assert abs(np.mean(np.abs(f) < 0.02) - 0.6827) < 0.01
    assert not np.array_equal(a[:1000], normal_bf16(5, 18, (1000,), 0.02))
