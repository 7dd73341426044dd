"""edgefm_prefill_tokens: the cache rows of given (prompt) tokens computed from the weights by the step kernel, one or two
tokens per call (Eq. 3 of the paper: KV <- Prefill(x); here for short suffixes behind a given prefix).  Oracle: the same tokens
stepped one by one."""
import numpy as np
import pytest

from edgefm_synth import CONFIGS, first_token
from helpers import Pair, assert_appended_rows_close, assert_logits_close, top2_margin, TOKEN_MARGIN

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("block_tokens,T0,n", [(2, 0, 9), (2, 20, 8), (0, 20, 5), (2, 64, 1)])
def test_prompt_tokens_through_the_step_kernel(block_tokens, T0, n):
    import torch
    cfg = CONFIGS["tiny"].with_(qkv_bias=True)
    pair = Pair(cfg, cache_len=T0, max_context=T0 + n + 3, block_tokens=block_tokens)
    try:
        rng = np.random.default_rng(100 + n)
        toks = rng.integers(0, cfg.vocab, n).tolist()
        pos0 = T0 + 11                                    # positions need not equal slots
        for i, t in enumerate(toks):
            ref_logits, ref_next = pair.oracle.step(t, pos0 + i)
        pair.ctx.prefill_tokens(toks, pos0)
        assert pair.ctx.cur_len == T0 + n == pair.oracle.cur_len      # exact on the host: every given token enters the cache
        torch.cuda.synchronize()
        assert pair.ctx.sync_length() == T0 + n
        kg, vg = [t.cpu().numpy().view(np.uint16) for t in pair.ctx.export_kv()]
        ko, vo = pair.oracle.export_kv()
        assert np.array_equal(kg[:, :, :T0], ko[:, :, :T0])
        assert_appended_rows_close(kg[:, :, T0:T0 + n], ko[:, :, T0:T0 + n])
        assert_appended_rows_close(vg[:, :, T0:T0 + n], vo[:, :, T0:T0 + n])
        # decoding continues from the device state: the greedy token after the last prompt token, the next position
        if top2_margin(ref_logits) > TOKEN_MARGIN:
            pair.ctx.step(-1, -1)
            torch.cuda.synchronize()
            ref2, _ = pair.oracle.step(ref_next, pos0 + n)
            assert_logits_close(pair.ctx.logits.cpu().numpy(), ref2, "first decode step after the prompt")
    finally:
        pair.close()


def test_prompt_longer_than_the_cache_is_rejected():
    from paper_2604_27476_b200 import EdgefmError, Status
    cfg = CONFIGS["tiny"]
    pair = Pair(cfg, cache_len=2, max_context=4, block_tokens=2)
    try:
        with pytest.raises(EdgefmError) as ei:
            pair.ctx.prefill_tokens([1, 2, 3], 2)
        assert ei.value.status == Status.ERR_CONTEXT_FULL and pair.ctx.cur_len == 2
        with pytest.raises(EdgefmError) as ei:
            pair.ctx.prefill_tokens([1, cfg.vocab], 2)
        assert ei.value.status == Status.ERR_INVALID_ARG
    finally:
        pair.close()
