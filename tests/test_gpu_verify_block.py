"""Block verification (Sec. 3.11 of the paper): two tokens pass through the step kernel in one call, the weights streamed
once.  The oracle verifies the block as the paper states it, token by token with plain decode steps; the draft model is not
part of either side, proposals are made here (the oracle's own greedy token = a proposal that must be accepted, anything
else = one that must be rejected)."""
import numpy as np
import pytest

from edgefm_synth import CONFIGS, first_token
from helpers import Pair, assert_logits_close, top2_margin, TOKEN_MARGIN

pytestmark = pytest.mark.gpu

SHAPES = {
    "tiny_d64": (CONFIGS["tiny"], 100),
    "d128_bias": (CONFIGS["tiny"].with_(hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn=1536, vocab=3000, n_layers=3, qkv_bias=True), 70),
    "ragged_g7": (CONFIGS["tiny"].with_(n_q_heads=7, n_kv_heads=1, hidden=136, ffn=72, vocab=333, n_layers=3, qkv_bias=True), 0),
    # the size and cache length bench.py --block-tokens 2 times
    "qwen2.5-1.5b_full_size": (CONFIGS["qwen2.5-1.5b"], CONFIGS["qwen2.5-1.5b"].cache_len),
}


def _peek_greedy(pair, tok, pos):
    """The oracle's greedy token after `tok`, without changing its cache."""
    n = pair.oracle.cur_len
    _, nxt = pair.oracle.step(tok, pos)
    pair.oracle.truncate(n)
    return nxt


@pytest.mark.parametrize("name", sorted(SHAPES))
def test_blocks_of_two_match_the_oracle_verification(name):
    import torch
    cfg, T0 = SHAPES[name]
    rounds = 8 if cfg.n_layers < 8 else 4
    pair = Pair(cfg, cache_len=T0, max_context=T0 + 2 * rounds + 2, block_tokens=2)
    try:
        tok, pos = first_token(cfg), T0 + 5
        for r in range(rounds):
            good = _peek_greedy(pair, tok, pos)
            proposal = good if r % 3 != 1 else (good + 1 + r) % cfg.vocab          # every third round: a wrong proposal
            ref_logits, ref_acc, ref_next = pair.oracle.verify_block([tok, proposal], pos)
            pair.ctx.verify_block([tok if r % 2 == 0 else -1, proposal], pos if r % 2 == 0 else -1)   # odd rounds: chained on the device
            torch.cuda.synchronize()
            got = pair.ctx.block_logits.cpu().numpy()
            assert_logits_close(got[0], ref_logits[0], f"{name} round {r} token 0")
            assert_logits_close(got[1], ref_logits[1], f"{name} round {r} token 1")
            assert int(pair.ctx.n_accepted.item()) == ref_acc == (2 if proposal == good else 1)
            margins_ok = all(top2_margin(ref_logits[t]) > TOKEN_MARGIN for t in range(ref_acc))
            if margins_ok:
                assert int(pair.ctx.next_token.item()) == ref_next
            assert pair.ctx.sync_length() == pair.oracle.cur_len
            tok, pos = ref_next, pos + ref_acc
            if not margins_ok:      # a near-tie: the two sides may legitimately continue with different tokens
                break
        # the cache: rows up to the common length agree with the oracle's (appended rows within one bf16 step)
        from helpers import assert_appended_rows_close
        n = pair.oracle.cur_len
        kg, vg = [t.cpu().numpy().view(np.uint16) for t in pair.ctx.export_kv()]
        ko, vo = pair.oracle.export_kv()
        assert np.array_equal(kg[:, :, :T0], ko[:, :, :T0]) and np.array_equal(vg[:, :, :T0], vo[:, :, :T0])
        if n > T0:
            assert_appended_rows_close(kg[:, :, T0:n], ko[:, :, T0:n])
            assert_appended_rows_close(vg[:, :, T0:n], vo[:, :, T0:n])
    finally:
        pair.close()


def test_plain_steps_and_single_token_blocks_on_a_block_context():
    """edgefm_decode_step and m = 1 blocks on a context built for blocks give the plain step's results."""
    import torch
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, cache_len=64, max_context=80, block_tokens=2)
    try:
        tok, pos = first_token(cfg), 64
        for s in range(4):
            ref, nxt = pair.oracle.step(tok, pos)
            if s % 2 == 0:
                pair.ctx.step(tok, pos)
            else:
                pair.ctx.verify_block([tok], pos)
            torch.cuda.synchronize()
            assert_logits_close(pair.ctx.logits.cpu().numpy(), ref, f"step {s}")
            if s % 2 == 1:
                assert int(pair.ctx.n_accepted.item()) == 1
            tok, pos = nxt, pos + 1
        assert pair.ctx.sync_length() == pair.oracle.cur_len == 68
    finally:
        pair.close()


def test_block_calls_are_validated():
    from paper_2604_27476_b200 import EdgefmError, Status, edgefm_create
    cfg = CONFIGS["tiny"]
    plain = Pair(cfg, cache_len=0, max_context=4)
    block = Pair(cfg, cache_len=3, max_context=4, block_tokens=2)
    try:
        with pytest.raises(EdgefmError) as ei:
            plain.ctx.verify_block([-1, 2], -1)                    # a plain context verifies through the dense path: tokens must be given
        assert ei.value.status == Status.ERR_INVALID_ARG
        with pytest.raises(EdgefmError) as ei:
            block.ctx.verify_block(list(range(1, 10)), 3)          # more than eight tokens
        assert ei.value.status == Status.ERR_INVALID_ARG
        with pytest.raises(EdgefmError) as ei:
            block.ctx.verify_block([1, 2, 3], 3)                   # the dense path for three tokens, one free slot
        assert ei.value.status == Status.ERR_CONTEXT_FULL
        with pytest.raises(EdgefmError) as ei:
            block.ctx.verify_block([1, cfg.vocab], 3)
        assert ei.value.status == Status.ERR_INVALID_ARG
        with pytest.raises(EdgefmError) as ei:
            block.ctx.verify_block([1, 2], 3)                      # one free slot, two tokens
        assert ei.value.status == Status.ERR_CONTEXT_FULL
        assert block.ctx.cur_len == 3
        shape = dict(n_layers=cfg.n_layers, hidden=cfg.hidden, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads, head_dim=cfg.head_dim,
                     ffn=cfg.ffn, vocab=cfg.vocab, rms_eps=cfg.rms_eps, rope_theta=cfg.rope_theta, qkv_bias=0)
        with pytest.raises(EdgefmError) as ei:
            edgefm_create(shape, plain.ptrs, 16, kv_format="int8", block_tokens=2)
        assert ei.value.status == Status.ERR_BAD_SHAPE
        with pytest.raises(EdgefmError) as ei:
            edgefm_create(shape, plain.ptrs, 9000, block_tokens=2)
        assert ei.value.status == Status.ERR_BAD_SHAPE
        with pytest.raises(EdgefmError) as ei:
            edgefm_create(shape, plain.ptrs, 16, block_tokens=3)                 # 0, 1, 2 or 4
        assert ei.value.status == Status.ERR_INVALID_ARG
    finally:
        plain.close(); block.close()


def test_block_verification_over_a_pruned_vocabulary():
    """With edgefm_set_vocab_subset the greedy tokens of a block, and with them the acceptance, are taken over the subset."""
    import torch
    from oracle import binding as O
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, cache_len=30, max_context=40, block_tokens=2)
    try:
        ids = np.unique(np.linspace(3, cfg.vocab - 1, 300).astype(np.int32))
        pair.ctx.set_vocab_subset(ids)
        tok, pos = int(ids[5]), 30
        for r in range(3):
            n0 = pair.oracle.cur_len
            l0, _ = pair.oracle.step(tok, pos)
            sub0, g0 = O.restricted_greedy(l0, ids)
            proposal = g0 if r != 1 else int(ids[(int(np.searchsorted(ids, g0)) + 1) % ids.size])
            l1, _ = pair.oracle.step(proposal, pos + 1)
            sub1, g1 = O.restricted_greedy(l1, ids)
            n_acc = 2 if proposal == g0 else 1
            pair.oracle.truncate(n0 + n_acc)
            pair.ctx.verify_block([tok, proposal], pos)
            torch.cuda.synchronize()
            got = pair.ctx.block_logits.cpu().numpy().reshape(-1)[:2 * ids.size].reshape(2, ids.size)   # rows of the subset's length
            assert_logits_close(got[0], sub0, f"round {r} token 0")
            assert_logits_close(got[1], sub1, f"round {r} token 1")
            assert int(pair.ctx.n_accepted.item()) == n_acc
            nxt = g1 if n_acc == 2 else g0
            if top2_margin(sub0) > TOKEN_MARGIN and (n_acc == 1 or top2_margin(sub1) > TOKEN_MARGIN):
                assert int(pair.ctx.next_token.item()) == nxt
            assert pair.ctx.sync_length() == pair.oracle.cur_len
            tok, pos = nxt, pos + n_acc
    finally:
        pair.close()


def _peek_chain(pair, tok, pos, k):
    """The oracle's next k greedy tokens after `tok`, without changing its cache."""
    n = pair.oracle.cur_len
    out = []
    for i in range(k):
        _, tok = pair.oracle.step(tok, pos + i)
        out.append(tok)
    pair.oracle.truncate(n)
    return out


@pytest.mark.parametrize("name", ["tiny_d64", "d128_bias", "qwen2.5-1.5b_full_size"])
def test_blocks_of_four_match_the_oracle_verification(name):
    """The four-token build (two bf16 pieces per activation): the first wrong proposal ends the block wherever it stands."""
    import torch
    cfg, T0 = SHAPES[name]
    rounds = 8 if cfg.n_layers < 8 else 4
    pair = Pair(cfg, cache_len=T0, max_context=T0 + 4 * rounds + 4, block_tokens=4)
    try:
        tok, pos = first_token(cfg), T0 + 2
        for r in range(rounds):
            props = _peek_chain(pair, tok, pos, 3)
            wrong_at = r % 4                                   # 0: none wrong; 1..3: proposal wrong_at is wrong
            if wrong_at:
                props[wrong_at - 1] = (props[wrong_at - 1] + 7) % cfg.vocab
            block = [tok] + props
            m = 4 if r != 5 else 3                             # once a shorter block
            block = block[:m]
            ref_logits, ref_acc, ref_next = pair.oracle.verify_block(block, pos)
            assert ref_acc == (min(wrong_at, m) if wrong_at else m)
            pair.ctx.verify_block([tok if r % 2 == 0 else -1] + block[1:], pos if r % 2 == 0 else -1)
            torch.cuda.synchronize()
            got = pair.ctx.block_logits.cpu().numpy()
            for t in range(m):
                assert_logits_close(got[t], ref_logits[t], f"{name} round {r} token {t}")
            assert int(pair.ctx.n_accepted.item()) == ref_acc
            assert pair.ctx.sync_length() == pair.oracle.cur_len
            if not all(top2_margin(ref_logits[t]) > TOKEN_MARGIN for t in range(ref_acc)):
                break
            assert int(pair.ctx.next_token.item()) == ref_next
            tok, pos = ref_next, pos + ref_acc
        from helpers import assert_appended_rows_close
        n = pair.oracle.cur_len
        kg, vg = [t.cpu().numpy().view(np.uint16) for t in pair.ctx.export_kv()]
        ko, vo = pair.oracle.export_kv()
        if n > T0:
            assert_appended_rows_close(kg[:, :, T0:n], ko[:, :, T0:n])
            assert_appended_rows_close(vg[:, :, T0:n], vo[:, :, T0:n])
    finally:
        pair.close()


@pytest.mark.parametrize("name,kv_format", [("tiny", None), ("tiny", "int8"), ("qwen2.5-1.5b", None)])
def test_blocks_of_up_to_eight_tokens_through_the_dense_path(name, kv_format):
    """Blocks longer than the context's block_tokens (here a plain context) are verified by the prefill kernels: all m tokens
    through the layers together, one pass over the output matrix for all rows, the acceptance rule on the device."""
    import torch
    cfg = CONFIGS[name] if name != "tiny" else CONFIGS[name].with_(qkv_bias=True)
    T0 = 40
    pair = Pair(cfg, cache_len=T0, max_context=T0 + 64, kv_format=kv_format)
    try:
        rng = np.random.default_rng(17)
        tok, pos = int(rng.integers(0, cfg.vocab)), T0 + 5
        for rnd, (m, wrong_at) in enumerate([(8, None), (8, 3), (5, 1), (7, 6), (6, None)]):
            # proposals: the oracle's own greedy continuation (found on a scratch pass, then rolled back), one of them spoiled
            start = pair.oracle.cur_len
            block, t = [tok], tok
            for i in range(m - 1):
                _, t = pair.oracle.step(t, pos + i)
                block.append(t)
            pair.oracle.truncate(start)
            if wrong_at is not None:
                block[wrong_at] = (block[wrong_at] + 1) % cfg.vocab
            ref_rows, ref_acc, ref_next = pair.oracle.verify_block(block, pos)
            pair.ctx.verify_block(block, pos)
            torch.cuda.synchronize()
            pair.ctx.sync_status()
            got = pair.ctx.block_logits.cpu().numpy()
            margins_ok = all(top2_margin(ref_rows[i]) > TOKEN_MARGIN for i in range(ref_acc))
            for i in range(ref_acc):
                assert_logits_close(got[i], ref_rows[i], f"round {rnd} row {i}")
            length = pair.ctx.sync_length()            # the host learns how far the cache grew (needed before the next long block)
            if not margins_ok:
                break                                  # a near-tie among the accepted rows: the two sides may decide differently
            assert int(pair.ctx.n_accepted.item()) == ref_acc, (rnd, int(pair.ctx.n_accepted.item()), ref_acc)
            assert length == pair.oracle.cur_len == start + ref_acc
            assert int(pair.ctx.next_token.item()) == ref_next
            tok, pos = ref_next, pos + ref_acc
        # without edgefm_sync_length the next long block is refused; -1 tokens are refused on this path
        from paper_2604_27476_b200 import EdgefmError, Status
        pair.ctx.verify_block([1, 2, 3, 4, 5], pos)
        with pytest.raises(EdgefmError) as ei:
            pair.ctx.verify_block([1, 2, 3, 4, 5], pos)
        assert ei.value.status == Status.ERR_INVALID_ARG
        pair.ctx.sync_length()
        with pytest.raises(EdgefmError) as ei:
            pair.ctx.verify_block([-1, 2, 3, 4, 5], pos)
        assert ei.value.status == Status.ERR_INVALID_ARG
        with pytest.raises(EdgefmError) as ei:
            pair.ctx.verify_block(list(range(1, 10)), pos)
        assert ei.value.status == Status.ERR_INVALID_ARG
    finally:
        pair.close()


def test_dense_block_with_a_pruned_output_layer():
    """The dense path on a context whose output layer is pruned: greedy tokens and acceptance are taken over the subset (here every
    second id plus the oracle's own choices, so that the oracle's unrestricted verification stays the reference)."""
    import torch
    cfg = CONFIGS["tiny"].with_(qkv_bias=True)
    T0 = 24
    pair = Pair(cfg, cache_len=T0, max_context=T0 + 16)
    try:
        tok, pos, m = 17, T0 + 2, 6
        start = pair.oracle.cur_len
        block, t = [tok], tok
        for i in range(m - 1):
            _, t = pair.oracle.step(t, pos + i)
            block.append(t)
        pair.oracle.truncate(start)
        block[4] = (block[4] + 1) % cfg.vocab                       # the fifth token is a wrong proposal
        ref_rows, ref_acc, ref_next = pair.oracle.verify_block(block, pos)
        greedy = [int(np.argmax(ref_rows[i])) for i in range(m)]
        ids = sorted(set(range(0, cfg.vocab, 2)) | set(greedy) | set(block))
        pair.ctx.set_vocab_subset(ids)
        pair.ctx.verify_block(block, pos)
        torch.cuda.synchronize()
        pair.ctx.sync_status()
        got = pair.ctx.block_logits.cpu().numpy().reshape(-1)[:m * len(ids)].reshape(m, len(ids))
        for i in range(ref_acc):
            assert_logits_close(got[i], ref_rows[i][ids], f"row {i}, pruned")
        if all(top2_margin(ref_rows[i]) > TOKEN_MARGIN for i in range(ref_acc)):
            assert int(pair.ctx.n_accepted.item()) == ref_acc == 4
            assert int(pair.ctx.next_token.item()) == ref_next
            assert pair.ctx.sync_length() == start + ref_acc
    finally:
        pair.close()
