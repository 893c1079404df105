"""The head-projection variant of the token mixer (Eq. 10) on the device against the oracle: q = W_in LN1(x),
heads of q mixed (recurrent form in decode, sequence-parallel form in prefill), x += W_out (.)."""
import dataclasses

import numpy as np
import pytest
import torch

import srm_inputs as I
from helpers import oracle_for, rel_err_rows
from parity import DEV, assert_greedy_coverage, teacher_forced

pytestmark = pytest.mark.gpu


def _build(shape, **kw):
    import paper_2605_08696_b200 as P
    W = I.make_weights(shape)
    return W, P.SRM(shape, W, device=DEV, **kw)


def test_tiny_fp32_with_head_projections_full_parity():
    shape = dataclasses.replace(I.CONFIGS["tiny"], head_proj=True)
    W, model = _build(shape)
    r = teacher_forced("tiny", shape, W, model, I.make_prompts("tiny"), 24)
    assert r["guarded"] == 0 and r["plain_mismatches"] == 0 and r["worst"] < 1e-4
    assert_greedy_coverage(r, 0.0)


@pytest.mark.parametrize("state_dtype", ["fp32", "bf16"])
def test_bf16_with_head_projections_parity_subset(state_dtype):
    shape = I.SRMShape(n_layers=4, d_model=512, vocab=8000, n_ctx=128, dtype="bf16", seed=21, head_proj=True)
    W, model = _build(shape, state_dtype=state_dtype)
    prompts = I.uniform_prompts(12, 50, shape.vocab, seed=8)      # 50 positions: six full tiles and a ragged one
    # (error bound of the small configuration; 72 decisions: a handful of guarded ones is a large share)
    r = teacher_forced("small" if state_dtype == "fp32" else "small/bf16-cache", shape, W, model, prompts, 6)
    assert_greedy_coverage(r, 0.12)


def test_head_projection_prefill_equals_decode_on_device_and_chunking():
    """Sequence-parallel prefill of n tokens leaves the cache and logits that n recurrent steps leave, and the
    result does not depend on how the batch is split into workspace passes."""
    import paper_2605_08696_b200 as P
    shape = I.SRMShape(n_layers=3, d_model=1024, vocab=2048, n_ctx=64, dtype="bf16", seed=22, head_proj=True)
    W, model = _build(shape)
    B, n = 40, 37
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=9)).to(DEV)
    g = P.Sampling("greedy")
    ws = model.new_workspace(B, n, prefill_samples=B)
    st_p = model.new_state(B)
    _, lg_p = model.prefill(st_p, prompts, g, ws, want_logits=True)
    st_r = model.new_state(B)
    for t in range(n):
        _, lg_r = model.decode_step(st_r, prompts[:, t].contiguous(), g, 0, ws, want_logits=True)
    assert rel_err_rows(lg_p.cpu().numpy(), lg_r.cpu().numpy()) < 2e-2
    assert rel_err_rows(st_p.cache().cpu().numpy(), st_r.cache().cpu().numpy()) < 2e-2
    ws_small = model.new_workspace(7, n, prefill_samples=3)
    st_c = model.new_state(B)
    _, lg_c = model.prefill(st_c, prompts, g, ws_small, want_logits=True)
    assert torch.equal(lg_c, lg_p) and torch.equal(st_c.cache(), st_p.cache())
    t1 = model.decode_step(st_c, None, g, 1, ws_small)
    t2 = model.decode_step(st_p, None, g, 1, ws)
    assert torch.equal(t1, t2)
    assert st_p.status() == 0 and st_r.status() == 0 and st_c.status() == 0


def test_weight_blob_layout_with_head_projections():
    import paper_2605_08696_b200 as P
    shape = dataclasses.replace(I.CONFIGS["tiny"], head_proj=True)
    W, model = _build(shape)
    base = P.SRM(I.CONFIGS["tiny"], I.make_weights(I.CONFIGS["tiny"]), device=DEV)
    assert model.blob.numel() == base.blob.numel() + 2 * 2 * 64 * 64 * 4
    assert torch.equal(model.tensor(1, 15).cpu(), torch.from_numpy(W["layers"][1]["W_in"]))
    assert torch.equal(model.tensor(1, 16).cpu(), torch.from_numpy(W["layers"][1]["W_out"]))
