"""Top-k / temperature / Philox selection fused into the LM head (no logits in HBM): the candidates of a row
are the logits at or above a threshold carried from the sample's previous selection; rows that cannot be settled
from their candidates are handed back to the logits path. Whatever happens to a row, its token must be the one
the logits path selects (which the other tests hold against the oracle's sampler), bit for bit."""
import numpy as np
import pytest
import torch

import srm_inputs as I
from helpers import weights_for

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _pair(shape, W):
    import paper_2605_08696_b200 as P
    return (P.SRM(shape, W, device=DEV, flags=P.FLAG_NO_SMALL_BATCH),
            P.SRM(shape, W, device=DEV, flags=P.FLAG_NO_FUSED_TOPK | P.FLAG_NO_SMALL_BATCH))


@pytest.mark.parametrize("B,k,T", [(300, 50, 0.8), (70, 1, 1.0), (257, 160, 0.7), (33, 7, 1.3)])
def test_fused_topk_generation_equals_the_logits_path(B, k, T):
    """Free-running generation through srm_generate, fused against unfused: same ids at every step, same cache.
    After the first step (no thresholds yet: every row is handed back) almost no row is."""
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["small"]                                    # L8 d512 V8000 bf16
    fused, plain = _pair(shape, weights_for("small"))
    n, gen = 16, 12
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=51)).to(DEV)
    samp = P.Sampling("topk", k, T, seed=1234, sample_idx_base=10_000)
    out = {}
    for name, model in (("fused", fused), ("plain", plain)):
        st = model.new_state(B)
        ws = model.new_workspace(B, n, prefill_samples=B)
        first = model.prefill(st, prompts, samp, ws)
        thr0 = st.topk_thresholds().clone()
        rest = model.generate(st, gen, 1, samp, ws)
        out[name] = (first.clone(), rest.clone(), st.cache().clone(), st.topk_handed_back(), thr0, st.topk_thresholds().clone())
        assert st.status() == 0
    assert torch.equal(out["fused"][0], out["plain"][0])
    assert torch.equal(out["fused"][1], out["plain"][1])
    assert torch.equal(out["fused"][2], out["plain"][2])
    assert out["plain"][3] == 0
    # the prefill's selection left a threshold for every row, so even the first decode step is settled from the
    # candidates; over 12 steps only a few rows may fall outside [k, 1024] candidates
    assert (out["fused"][4].view(torch.int32) != 0).all()
    assert out["fused"][3] <= max(2, 0.01 * B * gen), out["fused"][3]
    assert len(set(out["fused"][1][:, -1].tolist())) > 1 or B == 1


def test_rows_without_usable_threshold_are_handed_back_and_still_exact():
    """Thresholds forced to 'none' (0 bits, NaN), far too high (no candidate) and far too low (more candidates than a
    list holds) before a step: every such row goes through the logits path inside the same call, and all ids
    equal those of the unfused model; the call leaves fresh thresholds."""
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["small"]
    fused, plain = _pair(shape, weights_for("small"))
    B, n = 200, 8
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=52)).to(DEV)
    samp = P.Sampling("topk", 50, 0.8, seed=77, sample_idx_base=5)
    st_f, st_p = fused.new_state(B), plain.new_state(B)
    ws = fused.new_workspace(B, n, prefill_samples=B)
    assert torch.equal(fused.prefill(st_f, prompts, samp, ws), plain.prefill(st_p, prompts, samp, ws))
    thr = st_f.topk_thresholds()
    good = thr.clone()
    thr[0:40] = 0.0
    thr[40:80] = float("nan")
    thr[80:120] = 1e30
    thr[120:160] = -1e30
    for step in (1, 2):
        tf = fused.decode_step(st_f, None, samp, step, ws)
        tp = plain.decode_step(st_p, None, samp, step, ws)
        assert torch.equal(tf, tp)
        if step == 1:
            assert st_f.topk_handed_back() == 160
            new = st_f.topk_thresholds()
            assert torch.isfinite(new).all() and (new.view(torch.int32) != 0).all()
            assert (new - good).abs().max() < 1.0          # same scale as the thresholds the prefill left
    assert st_f.topk_handed_back() <= 162
    assert torch.equal(st_f.cache(), st_p.cache())
    assert st_f.status() == 0 and st_p.status() == 0


def test_fused_topk_in_workspace_sized_passes_and_with_the_token_store():
    """Several passes per step (a workspace for 96 rows, 250 samples): per-pass lists, counters and handed-back
    rows do not mix; tokens land in the right rows and columns of the store."""
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["small"]
    fused, plain = _pair(shape, weights_for("small"))
    B, n, gen = 250, 8, 6
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=53)).to(DEV)
    samp = P.Sampling("topk", 50, 0.8, seed=3, sample_idx_base=0)
    res = []
    for model, chunk in ((fused, 96), (plain, B)):
        st = model.new_state(B)
        ws = model.new_workspace(chunk, n, prefill_samples=chunk)
        model.prefill(st, prompts, samp, ws)
        store = torch.full((B, gen + 2), -1, dtype=torch.int32, device=DEV)
        model.generate(st, gen, 1, samp, ws, out=store[:, 1:])
        res.append(store.clone())
        assert st.status() == 0
    assert torch.equal(res[0], res[1])
    assert (res[0][:, 0] == -1).all() and (res[0][:, -1] == -1).all() and (res[0][:, 1:-1] >= 0).all()


def test_k_above_the_fused_limit_takes_the_logits_path():
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["small"]
    fused, plain = _pair(shape, weights_for("small"))
    B, n = 40, 8
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=54)).to(DEV)
    samp = P.Sampling("topk", 200, 0.9, seed=8, sample_idx_base=1)
    st_f, st_p = fused.new_state(B), plain.new_state(B)
    ws = fused.new_workspace(B, n, prefill_samples=B)
    fused.prefill(st_f, prompts, samp, ws); plain.prefill(st_p, prompts, samp, ws)
    for step in (1, 2, 3):
        assert torch.equal(fused.decode_step(st_f, None, samp, step, ws), plain.decode_step(st_p, None, samp, step, ws))
    assert st_f.topk_handed_back() == 0


def test_fused_topk_on_the_rollout_model_equals_the_logits_path_over_many_steps():
    """The rl model (L24 d1536 V32000), replicas of two prompts, 96 free-running sampled steps: thresholds carried
    from step to step on nearly flat logits; every id equal to the logits path, and after the prefill's thresholds
    only a few rows per thousand decisions are handed back."""
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["rl"]
    fused, plain = _pair(shape, weights_for("rl"))
    reps, n, gen = 12, 200, 96
    base = torch.from_numpy(I.make_prompts("rl", batch=32)[::2][:2].copy()).to(DEV)      # two distinct prompts
    B = 2 * reps
    samp = P.Sampling("topk", 50, 0.8, seed=shape.seed, sample_idx_base=4096)
    outs = []
    for model in (fused, plain):
        st = model.new_state(B)
        ws = model.new_workspace(B, n, prefill_samples=4)
        first = model.prefill_replicated(st, base, reps, samp, ws)
        rest = model.generate(st, gen, 1, samp, ws)
        outs.append((first.clone(), rest.clone(), st.topk_handed_back()))
        assert st.status() == 0
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    assert outs[1][2] == 0 and outs[0][2] <= 0.01 * B * gen, outs[0][2]
    assert len({tuple(r.tolist()) for r in outs[0][1][:reps]}) == reps                    # replicas of one prompt diverge


@pytest.mark.parametrize("scale", [8.0, 0.05])
def test_fused_topk_stays_exact_when_the_logit_scale_is_far_from_the_random_init_one(scale):
    """An LM head scaled up (peaked distributions: a few logits far above the rest, candidate counts that swing
    from step to step) or down (all logits within a hair of each other): whatever the carried thresholds do, rows
    outside [k, 1024] candidates are handed back and every id equals the logits path."""
    import copy
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["small"]
    W = copy.copy(weights_for("small"))
    W["W_lm"] = I.round_to_bf16(W["W_lm"] * np.float32(scale))
    fused, plain = _pair(shape, W)
    B, n, gen = 120, 12, 16
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=55)).to(DEV)
    samp = P.Sampling("topk", 40, 0.9, seed=17, sample_idx_base=77)
    outs = []
    for model in (fused, plain):
        st = model.new_state(B)
        ws = model.new_workspace(B, n, prefill_samples=B)
        first = model.prefill(st, prompts, samp, ws)
        rest = model.generate(st, gen, 1, samp, ws)
        outs.append((first.clone(), rest.clone(), st.topk_handed_back()))
        assert st.status() == 0
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    assert outs[0][2] <= 0.25 * B * gen, outs[0][2]          # (exactness never depends on it; this bounds the cost)
