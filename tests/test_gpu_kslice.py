"""Small decode passes: the down projection with its K dimension cut into ranges (one CTA pair per tile and range,
partial products in planes that the next layer's mixer and the final norm add in a fixed order). Same products,
another order of fp32 additions: logits and cache must agree with the whole-tile path to fp32 rounding through
bf16 layers, tokens wherever the decision is not thin, and rows must not depend on the batch they are in."""
import numpy as np
import pytest
import torch

import srm_inputs as I
from helpers import custom_shape, rel_err_rows, top2_margin, oracle_for

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("B,d,state_dtype", [(1, 512, "fp32"), (100, 512, "fp32"), (300, 1024, "fp16"), (700, 1536, "fp32"),
                                             (1100, 1024, "fp32")])
def test_ranges_of_k_agree_with_whole_tiles_and_with_the_oracle(B, d, state_dtype):
    import paper_2605_08696_b200 as P
    shape = custom_shape(n_layers=3, d_model=d, vocab=2048, n_ctx=24, dtype="bf16", seed=9)
    W = I.make_weights(shape)
    rng = np.random.default_rng(B)
    prompts_np = rng.integers(0, shape.vocab, size=(B, 5)).astype(np.int32)
    prompts = torch.from_numpy(prompts_np).to(DEV)
    outs, fed = [], None                                       # the second run consumes the first run's tokens
    for flags in (P.FLAG_NO_SMALL_BATCH, P.FLAG_NO_SMALL_BATCH | P.FLAG_NO_KSLICE):
        m = P.SRM(shape, W, device=DEV, flags=flags, state_dtype=state_dtype)
        st = m.new_state(B)
        ws = m.new_workspace(B, 5, prefill_samples=B)
        samp = P.Sampling("greedy")
        tok, lg0 = m.prefill(st, prompts, samp, ws, want_logits=True)
        lgs, toks = [lg0.clone()], [tok.clone()]
        for k in range(4):
            tok, lg = m.decode_step(st, tok if fed is None else fed[k], samp, k + 1, ws, want_logits=True)
            lgs.append(lg.clone()); toks.append(tok.clone())
        assert st.status() == 0
        fed = fed if fed is not None else [t.clone() for t in toks]
        outs.append((torch.stack(lgs).cpu().numpy(), torch.stack(toks).cpu().numpy(), st.cache().float().cpu().numpy()))
    (lg_a, tok_a, S_a), (lg_b, tok_b, S_b) = outs
    assert not np.array_equal(lg_a[1:], lg_b[1:])            # (the ranges did run: another order of additions)
    assert np.array_equal(lg_a[0], lg_b[0])                  # (the prefill is the same path)
    assert rel_err_rows(lg_a, lg_b) < 4e-3 and rel_err_rows(S_a, S_b) < 4e-3
    differ = tok_a != tok_b
    assert np.all(top2_margin(lg_b)[differ] < 1e-2)
    # the path with ranges against the oracle, teacher-forced with the device's own tokens
    n_chk = min(B, 16)
    orc = oracle_for(shape, W)
    lo, state = orc.forward_parallel(prompts_np[:n_chk])
    assert rel_err_rows(lg_a[0][:n_chk], lo[:, -1]) < 3e-2
    for k in range(4):
        lo, state = orc.decode_step(state, tok_a[k][:n_chk], 5 + k)
        assert rel_err_rows(lg_a[k + 1][:n_chk], lo) < 3e-2


def test_rows_do_not_depend_on_the_batch_or_the_workspace_they_are_in():
    """The number of ranges depends on the tile count only, and the planes have room of their own in the workspace:
    a row gives the same bits alone, in a batch of 200 and in that batch processed in passes of 64."""
    import paper_2605_08696_b200 as P
    shape = custom_shape(n_layers=3, d_model=512, vocab=1024, n_ctx=24, dtype="bf16", seed=10)
    W = I.make_weights(shape)
    prompts = torch.from_numpy(np.random.default_rng(2).integers(0, shape.vocab, size=(200, 4)).astype(np.int32)).to(DEV)
    m = P.SRM(shape, W, device=DEV, flags=P.FLAG_NO_SMALL_BATCH)
    res = []
    for B, chunk in [(200, 200), (200, 64), (3, 3)]:
        st = m.new_state(B)
        ws = m.new_workspace(chunk, 4, prefill_samples=chunk)
        tok, _ = m.prefill(st, prompts[:B], P.Sampling("greedy"), ws, want_logits=True)
        for k in range(3):
            tok, lg = m.decode_step(st, tok, P.Sampling("greedy"), k + 1, ws, want_logits=True)
        assert st.status() == 0
        res.append((lg.clone(), st.cache().clone()))
    assert torch.equal(res[0][0], res[1][0]) and torch.equal(res[0][1], res[1][1])
    assert torch.equal(res[0][0][:3], res[2][0]) and torch.equal(res[0][1][:, :3], res[2][1])
