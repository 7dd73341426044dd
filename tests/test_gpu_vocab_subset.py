"""Vocabulary pruning of the output layer (caption of Fig. 2): the CUDA step restricted to a subset of token ids
against the oracle's logits restricted to the same ids.

The oracle computes the full logits; `restricted_greedy` keeps the subset's entries and takes the greedy choice
among them.  The CUDA path gathers the subset's rows once and streams only those.
"""
import numpy as np
import pytest

from edgefm_synth import CONFIGS, first_token
from helpers import Pair, TOKEN_MARGIN, assert_logits_close, top2_margin

pytestmark = pytest.mark.gpu


def _subset(vocab, n, seed):
    rng = np.random.default_rng(seed)
    return np.sort(rng.choice(vocab, n, replace=False)).astype(np.int32)


def _check_step(pair, tok, pos, ids, what):
    """One step on both sides; compares the subset's logits and the restricted greedy token.  Returns the oracle's choice."""
    import torch
    from oracle import binding as O
    ref_logits, ref_full_next = pair.oracle.step(tok, pos)
    pair.ctx.step(tok, pos)
    torch.cuda.synchronize()
    if ids is None:
        gpu = pair.ctx.logits.cpu().numpy()
        ref, ref_next = ref_logits, ref_full_next
    else:
        gpu = pair.ctx.logits[: len(ids)].cpu().numpy()
        ref, ref_next = O.restricted_greedy(ref_logits, ids)
    assert_logits_close(gpu, ref, what)
    if len(ref) == 1 or top2_margin(ref) > TOKEN_MARGIN:
        assert int(pair.ctx.next_token.item()) == ref_next, what
    return ref_next


# sizes: one row, fewer rows than warps, fewer rows than CTAs, ragged counts around the tile and grid sizes, all rows
@pytest.mark.parametrize("n", [1, 7, 100, 148 * 12 + 5, 2049, 4095, 4096])
def test_tiny_subset_sizes(n):
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, max_context=cfg.cache_len + 8)
    try:
        ids = _subset(cfg.vocab, n, seed=n)
        pair.ctx.set_vocab_subset(ids)
        tok, pos = first_token(cfg), cfg.first_position
        for s in range(3):
            tok = _check_step(pair, tok, pos + s, ids, f"tiny subset {n} step {s}")
            assert tok in ids
    finally:
        pair.close()


def test_subset_switch_and_restore():
    """Full vocabulary -> subset A -> subset B (larger) -> full again, on one context, the cache growing throughout."""
    import torch
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, max_context=cfg.cache_len + 16)
    try:
        tok, pos = first_token(cfg), cfg.first_position
        plan = [None, _subset(cfg.vocab, 300, 1), _subset(cfg.vocab, 3000, 2), None, _subset(cfg.vocab, 5, 3)]
        step = 0
        for ids in plan:
            pair.ctx.set_vocab_subset(ids)
            for _ in range(2):
                tok = _check_step(pair, tok, pos + step, ids, f"plan step {step}")
                step += 1
        assert pair.ctx.cur_len == cfg.cache_len + step
        torch.cuda.synchronize()
    finally:
        pair.close()


def test_planted_maximum_outside_subset_is_ignored():
    """An lm_head row that wins by far over the full vocabulary must not win when it is not in the subset."""
    import torch
    from edgefm_synth import make_weights
    cfg = CONFIGS["tiny"]
    w = make_weights(cfg)
    pair0 = Pair(cfg, weights=w, max_context=cfg.cache_len + 4)
    try:
        tok, pos = first_token(cfg), cfg.first_position
        _, full_next = pair0.oracle.step(tok, pos)
    finally:
        pair0.close()
    ids = np.array([t for t in range(0, cfg.vocab, 3) if t != full_next], np.int32)
    pair = Pair(cfg, weights=w, max_context=cfg.cache_len + 4)
    try:
        pair.ctx.set_vocab_subset(ids)
        nxt = _check_step(pair, tok, pos, ids, "winner outside the subset")
        assert nxt != full_next
        torch.cuda.synchronize()
    finally:
        pair.close()


def test_subset_device_chaining():
    """Steps chained on the device (token -1) under a subset feed the chosen full-vocabulary id back in."""
    import torch
    from oracle import binding as O
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, max_context=cfg.cache_len + 8)
    try:
        ids = _subset(cfg.vocab, 1500, 9)
        pair.ctx.set_vocab_subset(ids)
        tok, pos = first_token(cfg), cfg.first_position
        pair.ctx.step(tok, pos)
        for _ in range(4):
            pair.ctx.step(-1, -1)
        torch.cuda.synchronize()
        gpu_last = pair.ctx.logits[: len(ids)].cpu().numpy()
        margins_ok = True
        for s in range(5):
            ref_logits, _ = pair.oracle.step(tok, pos + s)
            ref, tok = O.restricted_greedy(ref_logits, ids)
            margins_ok = margins_ok and top2_margin(ref) > TOKEN_MARGIN
        if margins_ok:   # same token sequence on both sides, so the last step saw the same inputs
            assert_logits_close(gpu_last, ref, "chained subset steps")
            assert int(pair.ctx.next_token.item()) == tok
    finally:
        pair.close()


def test_subset_rejects_bad_ids():
    from paper_2604_27476_b200 import EdgefmError
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, max_context=cfg.cache_len + 4)
    try:
        good = _subset(cfg.vocab, 50, 4)
        pair.ctx.set_vocab_subset(good)
        for bad in ([5, 4, 9], [3, 3, 8], [-1, 2], [0, cfg.vocab]):
            with pytest.raises(EdgefmError):
                pair.ctx.set_vocab_subset(np.array(bad, np.int32))
        # the previous subset is still in force
        _check_step(pair, first_token(cfg), cfg.first_position, good, "after rejected subsets")
    finally:
        pair.close()


def test_subset_at_benchmark_size():
    """Qwen2.5-1.5B shape, 32768 of 151936 ids, at the full cache length: four steps."""
    cfg = CONFIGS["qwen2.5-1.5b"]
    pair = Pair(cfg, max_context=cfg.cache_len + 8)
    try:
        ids = _subset(cfg.vocab, 32768, 11)
        pair.ctx.set_vocab_subset(ids)
        tok, pos = first_token(cfg), cfg.first_position
        for s in range(4):
            tok = _check_step(pair, tok, pos + s, ids, f"1.5b subset step {s}")
    finally:
        pair.close()
