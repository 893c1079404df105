"""The single-kernel decode step of small batches (at most 64 samples; step_small.cuh): one cooperative kernel
runs embedding, every layer's cache update and feed-forward, the final norm, the LM head and the greedy selection,
with the projections cut into per-SM slabs. Parity against the oracle (teacher-forced: logits at every step, the
cache at the end, tokens under the margin rule), agreement with the kernel-per-operation path, sampling on the
logits it writes, and replay from a captured graph."""
import numpy as np
import pytest
import torch

import srm_inputs as I
from helpers import rel_err_rows, weights_for
from parity import DEV, assert_greedy_coverage, teacher_forced

pytestmark = pytest.mark.gpu


def _model(name, **kw):
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS[name]
    return shape, weights_for(name), P.SRM(shape, weights_for(name), device=DEV, **kw)


def _launches_of_one_step(model, st, samp, ws):
    import paper_2605_08696_b200 as P
    n0 = P.SRM.kernel_launches()
    model.decode_step(st, None, samp, 99, ws)
    return P.SRM.kernel_launches() - n0


@pytest.mark.parametrize("B,state_dtype", [(1, "fp32"), (8, "fp32"), (33, "fp16"), (64, "fp32"), (16, "bf16")])
def test_small_model_small_batch_parity(B, state_dtype):
    """L8 d512 V8000 (eight n-slabs x eight k-slabs in the down projection, 16-column slabs in the up
    projection, ragged last LM-head slab): 1 to 64 rows, partly filled row tiles included."""
    import paper_2605_08696_b200 as P
    shape, W, model = _model("small", state_dtype=state_dtype)
    prompts = I.make_prompts("small")[7:7 + B]
    key = "small" if state_dtype == "fp32" else "small/bf16-cache"
    r = teacher_forced(key, shape, W, model, prompts, 16)
    if B >= 8:
        assert_greedy_coverage(r, 0.10 if state_dtype != "bf16" else 0.25)
    # the step really was the single kernel: one launch for a greedy step without logits
    st = model.new_state(B)
    ws = model.new_workspace(B, 128, prefill_samples=B)
    model.prefill(st, torch.from_numpy(prompts).to(DEV), P.Sampling("greedy"), ws)
    assert _launches_of_one_step(model, st, P.Sampling("greedy"), ws) == 1
    assert st.status() == 0


def test_small_config_full_horizon_on_the_single_kernel_path():
    """128 + 384 tokens to the end of the context, 8 samples."""
    shape, W, model = _model("small")
    w = I.WORKLOADS["small"]
    prompts = I.make_prompts("small")[200:208]
    r = teacher_forced("small", shape, W, model, prompts, w["gen"], run_to_ctx_end=True)
    assert_greedy_coverage(r, 0.02)


def test_mid_model_small_batch_parity():
    """L16 d1024 V32000: 32-column slabs of the up projection, 512-long k-slabs, 224-column LM-head slabs."""
    shape, W, model = _model("mid")
    prompts = I.make_prompts("mid", batch=64)[3:11]
    r = teacher_forced("mid", shape, W, model, prompts, 10)
    assert_greedy_coverage(r, 0.15)


def test_single_kernel_step_agrees_with_the_kernel_per_operation_path():
    """Same sums in another order (slabs of K in the down projection, mma.sync fragments instead of tcgen05 tiles).
    Both paths consume the SAME tokens (those the kernel-per-operation path selects): logits agree to a fraction of
    the bf16 tolerance at every step, the cache likewise, and the selected tokens are equal wherever the top-2
    margin is not thin."""
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["small"]
    W = weights_for("small")
    small, big = P.SRM(shape, W, device=DEV), P.SRM(shape, W, device=DEV, flags=P.FLAG_NO_SMALL_BATCH)
    B, n = 48, 32
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=61)).to(DEV)
    g = P.Sampling("greedy")
    st_s, st_b = small.new_state(B), big.new_state(B)
    ws = big.new_workspace(B, n, prefill_samples=B)
    tok = big.prefill(st_b, prompts, g, ws)
    assert torch.equal(small.prefill(st_s, prompts, g, ws), tok)               # (the prefill is the same code on both)
    for k in range(8):
        tok_b, lg_b = big.decode_step(st_b, tok, g, k + 1, ws, want_logits=True)
        tok_s, lg_s = small.decode_step(st_s, tok, g, k + 1, ws, want_logits=True)
        lb, ls = lg_b.cpu().numpy(), lg_s.cpu().numpy()
        assert rel_err_rows(ls, lb) < 5e-3, k
        part = np.partition(lb, -2, axis=-1)
        safe = torch.from_numpy((part[..., -1] - part[..., -2]) > 2e-2).to(DEV)
        assert torch.equal(tok_s[safe], tok_b[safe])
        tok = tok_b
    assert rel_err_rows(st_s.cache().cpu().numpy(), st_b.cache().cpu().numpy()) < 5e-3
    assert st_s.status() == 0 and st_b.status() == 0


@pytest.mark.parametrize("mode", ["topk", "topp"])
def test_sampling_on_the_logits_of_the_single_kernel_step(mode):
    """Sampled selection: the kernel writes the logits, the selection kernels follow. The oracle's sampler run on
    those logits picks the device's token (CDF-edge cases excepted)."""
    import paper_2605_08696_b200 as P
    from oracle import srm_oracle as O
    from helpers import topp_is_strict
    shape, W, model = _model("small")
    B, n = 24, 16
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=62)).to(DEV)
    samp = P.Sampling("topk", 50, 0.8, seed=21, sample_idx_base=300) if mode == "topk" else \
        P.Sampling("topp", temperature=0.7, seed=21, sample_idx_base=300, top_p=0.9)
    st = model.new_state(B)
    ws = model.new_workspace(B, n, prefill_samples=B)
    model.prefill(st, prompts, samp, ws)
    checked = 0
    for k in range(1, 5):
        tok, lg = model.decode_step(st, None, samp, k, ws, want_logits=True)
        lg_np, t = lg.cpu().numpy(), tok.cpu().numpy()
        if mode == "topk":
            want, det = O.select_topk(lg_np, 50, 0.8, 21, 300 + np.arange(B), k, return_detail=True)
            for b in range(B):
                if want[b] != t[b]:
                    c, thr = det[b]["cdf"], det[b]["thr"]
                    assert np.min(np.abs(c - thr)) < 1e-6 * c[-1]
                else:
                    checked += 1
        else:
            want, det = O.select_topp(lg_np, np.float32(0.9), 0.7, 21, 300 + np.arange(B), k, return_detail=True)
            for b in range(B):
                if topp_is_strict(lg_np[b], float(np.float32(0.9)), 0.7, det[b]):
                    assert want[b] == t[b]
                    checked += 1
        # without logits: the same tokens (the logits then go to the workspace)
    assert checked > 0.9 * 4 * B and st.status() == 0


def test_generation_replayed_from_a_graph_equals_launch_by_launch_on_the_single_kernel_path():
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["small"]
    W = weights_for("small")
    B, n = 20, 24
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=63)).to(DEV)
    outs = []
    for flags in (P.FLAG_NO_GRAPH, P.FLAG_GRAPH):
        model = P.SRM(shape, W, device=DEV, flags=flags)
        for samp in (P.Sampling("greedy"), P.Sampling("topk", 50, 0.8, seed=4, sample_idx_base=9)):
            st = model.new_state(B)
            ws = model.new_workspace(B, n, prefill_samples=B)
            first = model.prefill(st, prompts, samp, ws)
            out = model.generate(st, 10, 1, samp, ws)
            out2 = model.generate(st, 6, 11, samp, ws, out=torch.empty(B, 6, dtype=torch.int32, device=DEV))
            assert st.pos == n + 16 and st.status() == 0
            outs.append((first.clone(), out.clone(), out2.clone(), st.cache().clone()))
    for a_, b_ in zip(outs[:2], outs[2:]):
        for x_, y_ in zip(a_, b_):
            assert torch.equal(x_, y_)


def test_batches_and_models_outside_the_single_kernel_path_are_unaffected():
    """65 samples, an fp32 model and a model with head projections take the kernel-per-operation path."""
    import dataclasses
    import paper_2605_08696_b200 as P
    shape, W, model = _model("small")
    g = P.Sampling("greedy")
    st = model.new_state(65)
    ws = model.new_workspace(65, 8, prefill_samples=65)
    model.prefill(st, torch.from_numpy(I.uniform_prompts(65, 8, shape.vocab, seed=64)).to(DEV), g, ws)
    assert _launches_of_one_step(model, st, g, ws) > 20
    tiny = I.CONFIGS["tiny"]
    mt = P.SRM(tiny, I.make_weights(tiny), device=DEV)
    st = mt.new_state(4)
    ws = mt.new_workspace(4, 8, prefill_samples=4)
    mt.prefill(st, torch.from_numpy(I.make_prompts("tiny")).to(DEV), g, ws)
    assert _launches_of_one_step(mt, st, g, ws) > 5
