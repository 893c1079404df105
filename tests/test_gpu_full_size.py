"""Parity at the full benchmark sizes, in the launch configuration bench.py times (full batch, same
workspace chunking): the device free-runs the whole batch; for rows sampled across the batch (first, last,
chunk boundaries) the oracle consumes the DEVICE's tokens, so its logits are comparable step by step.
Checked per sampled row and step: logits within the bf16 tolerance; the device's greedy token equals the
oracle's argmax wherever the oracle's margin exceeds 1e-2 and twice the row's logit error; for top-k / Philox
sampling the oracle's sampler applied to the device's logits picks the device's token. A second, logit-free
run (the fused selection path that bench.py times) must emit exactly the tokens of the first."""
import numpy as np
import pytest
import torch

import srm_inputs as I
from helpers import oracle_for, rel_err_rows, top2_margin, weights_for

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL, MARGIN = 3e-2, 1e-2


def _run(name, steps, rows, chunk):
    import paper_2605_08696_b200 as P
    from oracle import srm_oracle as O
    w = I.WORKLOADS[name]
    shape = I.CONFIGS[w["model"]]
    B, n = w["batch"], w["prompt_len"]
    W = weights_for(w["model"])
    model = P.SRM(shape, W, device=DEV)
    topk = w["sampling"] == "topk"
    samp = P.Sampling("topk", w["top_k"], w["temperature"], seed=shape.seed) if topk else P.Sampling("greedy")
    prompts_np = I.make_prompts(name)
    prompts = torch.from_numpy(prompts_np).to(DEV)
    ws = model.new_workspace(chunk, n, prefill_samples=max(1, 65536 // n))

    # ---- run 1: logits requested (LM head + selection kernel) ----
    st = model.new_state(B)
    tok, lg = model.prefill(st, prompts, samp, ws, want_logits=True)
    toks, logits = [tok.clone()], [lg[rows].cpu().numpy()]
    for k in range(1, steps):
        tok, lg = model.decode_step(st, None, samp, k, ws, want_logits=True)
        toks.append(tok.clone()); logits.append(lg[rows].cpu().numpy())
    assert st.status() == 0
    dev_tok = torch.stack(toks, 1)
    del lg

    # ---- run 2: no logits (greedy: selection fused into the LM head), the path bench.py times ----
    st2 = model.new_state(B)
    first2 = model.prefill(st2, prompts, samp, ws)
    rest2 = model.generate(st2, steps - 1, 1, samp, ws)
    assert torch.equal(torch.cat([first2[:, None], rest2], 1), dev_tok)
    assert st2.status() == 0

    # ---- oracle on the sampled rows, fed the device's tokens ----
    orc = oracle_for(shape, W)
    dt = dev_tok[rows].cpu().numpy()
    lg_o, state = orc.forward_parallel(prompts_np[rows])
    cur = lg_o[:, -1]
    checked = 0
    for k in range(steps):
        got = logits[k]
        assert rel_err_rows(got, cur) < TOL, (name, k, rel_err_rows(got, cur))
        if topk:
            pick = O.select_topk(got, w["top_k"], w["temperature"], shape.seed, np.asarray(rows), k, return_detail=True)
            for i, b in enumerate(rows):
                if pick[0][i] != dt[i, k]:
                    c, thr = pick[1][i]["cdf"], pick[1][i]["thr"]
                    assert np.min(np.abs(c - thr)) < 1e-6 * c[-1], (name, k, b)
                checked += 1
        else:
            eps = np.max(np.abs(got - cur), axis=-1)
            strict = top2_margin(cur) > np.maximum(MARGIN, 2 * eps)
            assert np.array_equal(dt[strict, k], O.select_greedy(cur)[strict]), (name, k)
            checked += int(strict.sum())
        if k + 1 < steps:
            cur, state = orc.decode_step(state, dt[:, k], n + k)
    assert checked > 0
    cache = torch.stack([st.layer(l)[rows].float() for l in range(shape.n_layers)]).cpu().numpy()
    assert rel_err_rows(cache, state) < TOL


def test_mid_full_batch_sampled_rows():
    """mid: L16 d1024 V32000 bf16, 4096 Zipf prompts of 256 tokens, greedy, one 4096-row pass per step."""
    _run("mid", steps=3, rows=[0, 1, 255, 256, 2047, 4000, 4095], chunk=4096)


def test_rl_full_batch_sampled_rows():
    """rl: L24 d1536 V32000 bf16, 16 prompts x 1024 replicas, top-k 50 / T 0.8 / Philox, 8192-row passes."""
    _run("rl", steps=2, rows=[0, 1023, 1024, 8191, 8192, 16383], chunk=8192)
