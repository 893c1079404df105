"""Prompts of different lengths in one batch (srm_prefill_ragged, then the ordinary step calls with one
position per sample kept on the device): every sample must behave as if it had been prefilled and decoded
alone. Checked against the oracle run sample by sample (each with its own length and positions), and against
the device's own single-sample runs."""
import numpy as np
import pytest
import torch

import srm_inputs as I
from helpers import oracle_for, rel_err_rows, top2_margin

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = {"fp32": 1e-4, "bf16": 3e-2}


def _ragged_batch(shape, lengths, seed):
    n_max = max(lengths)
    toks = I.uniform_prompts(len(lengths), n_max, shape.vocab, seed=seed)
    for b, n in enumerate(lengths):
        toks[b, n:] = (7 * b + 3) % shape.vocab           # padding: valid ids that must not matter
    return toks


@pytest.mark.parametrize("name,lengths,gen", [
    ("tiny", [8, 3, 5, 1, 8, 6], 12),                     # fp32, d 64: 1e-4
    ("small", [40, 17, 33, 9, 40, 1, 25], 6),             # bf16, d 512, several position tiles and a ragged last tile
])
def test_ragged_batch_matches_the_oracle_run_sample_by_sample(name, lengths, gen):
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS[name]
    W = I.make_weights(shape)
    model = P.SRM(shape, W, device=DEV)
    orc = oracle_for(shape, W)
    B, n_max = len(lengths), max(lengths)
    toks = _ragged_batch(shape, lengths, seed=17)
    st = model.new_state(B)
    ws = model.new_workspace(B, n_max, prefill_samples=B)
    g = P.Sampling("greedy")
    lens_dev = torch.tensor(lengths, dtype=torch.int32, device=DEV)
    tok, lg = model.prefill_ragged(st, torch.from_numpy(toks).to(DEV), lens_dev, g, ws, want_logits=True)
    assert st.pos == n_max
    # the oracle, one sample at a time, fed the device's tokens (teacher forcing)
    states = []
    worst, checked = 0.0, 0
    lg_np, tok_np = lg.cpu().numpy(), tok.cpu().numpy()
    for b, n in enumerate(lengths):
        lo, so = orc.forward_parallel(toks[b:b + 1, :n])
        worst = max(worst, rel_err_rows(lg_np[b], lo[0, n - 1]))
        if top2_margin(lo[0, n - 1]) > 1e-2 + 2 * np.max(np.abs(lg_np[b] - lo[0, n - 1])):
            assert tok_np[b] == int(np.argmax(lo[0, n - 1]))
            checked += 1
        states.append(so)
    for k in range(gen):
        tok_in = tok_np.copy()
        tok, lg = model.decode_step(st, None, g, k + 1, ws, want_logits=True)
        lg_np, tok_np = lg.cpu().numpy(), tok.cpu().numpy()
        for b, n in enumerate(lengths):
            lo, states[b] = orc.decode_step(states[b], tok_in[b:b + 1], n + k)      # this sample's own position
            worst = max(worst, rel_err_rows(lg_np[b], lo[0]))
            if top2_margin(lo[0]) > 1e-2 + 2 * np.max(np.abs(lg_np[b] - lo[0])):
                assert tok_np[b] == int(np.argmax(lo[0]))
                checked += 1
    assert worst < TOL[shape.dtype], worst
    assert checked > 0.5 * B * (gen + 1)
    cache = st.cache().cpu().numpy()
    for b in range(B):
        assert rel_err_rows(cache[:, b], states[b][:, 0]) < TOL[shape.dtype]
    assert st.pos == n_max + gen and st.status() == 0


@pytest.mark.parametrize("sampling", ["greedy", "topk"])
def test_ragged_batch_equals_single_sample_runs_on_the_device(sampling):
    """Same kernels, same arithmetic: sample b of the ragged batch and a batch of one holding only that prompt
    (same Philox sample index) give the same tokens and the same cache, bit for bit; the uniform API on that
    prompt agrees to rounding (it may take the streaming mixer kernel, whose LayerNorm sums run in another
    order)."""
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["small"]
    W = I.make_weights(shape)
    model = P.SRM(shape, W, device=DEV)
    lengths = [31, 8, 19, 31, 2]
    B, n_max, gen = len(lengths), max(lengths), 8
    toks = _ragged_batch(shape, lengths, seed=23)
    mk = (lambda base: P.Sampling("greedy")) if sampling == "greedy" else \
        (lambda base: P.Sampling("topk", 50, 0.8, seed=9, sample_idx_base=base))
    st = model.new_state(B)
    ws = model.new_workspace(B, n_max, prefill_samples=B)
    lens_dev = torch.tensor(lengths, dtype=torch.int32, device=DEV)
    first = model.prefill_ragged(st, torch.from_numpy(toks).to(DEV), lens_dev, mk(100), ws).clone()
    rest = model.generate(st, gen, 1, mk(100), ws)               # the generation loop (graph or launches) works on it too
    got = torch.cat([first[:, None], rest], 1).cpu().numpy()
    cache = st.cache()
    for b, n in enumerate(lengths):
        s1 = model.new_state(1)
        w1 = model.new_workspace(1, n, prefill_samples=1)
        t1 = torch.from_numpy(toks[b:b + 1, :n].copy()).to(DEV)
        f1 = model.prefill_ragged(s1, t1, lens_dev[b:b + 1].clone(), mk(100 + b), w1).clone()
        r1 = model.generate(s1, gen, 1, mk(100 + b), w1)
        alone = torch.cat([f1[:, None], r1], 1).cpu().numpy()[0]
        assert np.array_equal(got[b], alone), (b, got[b], alone)
        assert torch.equal(cache[:, b], s1.cache()[:, 0])
        assert s1.pos == n + gen
        # the uniform API on the same prompt: same first-token logits up to rounding
        s2 = model.new_state(1)
        _, lg_u = model.prefill(s2, t1, mk(100 + b), w1, want_logits=True)
        s3 = model.new_state(1)
        _, lg_r = model.prefill_ragged(s3, t1, lens_dev[b:b + 1].clone(), mk(100 + b), w1, want_logits=True)
        assert rel_err_rows(lg_r.cpu().numpy(), lg_u.cpu().numpy()) < 1e-3
    assert st.pos == n_max + gen and st.status() == 0


def test_ragged_with_head_projections_and_argument_checks():
    import dataclasses
    import paper_2605_08696_b200 as P
    shape = dataclasses.replace(I.CONFIGS["small"], head_proj=True)
    W = I.make_weights(shape)
    model = P.SRM(shape, W, device=DEV)
    orc = oracle_for(shape, W)
    lengths = [12, 5, 9]
    B, n_max = 3, 12
    toks = _ragged_batch(shape, lengths, seed=29)
    st = model.new_state(B)
    ws = model.new_workspace(B, n_max, prefill_samples=B)
    g = P.Sampling("greedy")
    lens_dev = torch.tensor(lengths, dtype=torch.int32, device=DEV)
    tok, lg = model.prefill_ragged(st, torch.from_numpy(toks).to(DEV), lens_dev, g, ws, want_logits=True)
    tok2, lg2 = model.decode_step(st, None, g, 1, ws, want_logits=True)
    for b, n in enumerate(lengths):
        lo, so = orc.forward_parallel(toks[b:b + 1, :n])
        assert rel_err_rows(lg.cpu().numpy()[b], lo[0, n - 1]) < 3e-2
        lo2, _ = orc.decode_step(so, tok.cpu().numpy()[b:b + 1], n)
        assert rel_err_rows(lg2.cpu().numpy()[b], lo2[0]) < 3e-2
    # positions live on the device now
    with pytest.raises(P.SRMError):
        st.pos = 3
    # a length outside [1, n_max] is clamped and reported
    st_bad = model.new_state(B)
    bad = torch.tensor([12, 0, 40], dtype=torch.int32, device=DEV)
    model.prefill_ragged(st_bad, torch.from_numpy(toks).to(DEV), bad, g, ws)
    assert st_bad.status() & 1


def test_ragged_prefill_through_the_scan_kernel_matches_the_tile_kernel():
    """With many prompts per pass the prefill mixer is the scan kernel, with few the tile kernel (explicit diagonal
    blocks of M): the same ragged prompts through both (one pass of 512 prompts, and passes of 64) leave the same
    cache and first tokens up to what bf16 activations allow (each kernel is checked against the oracle elsewhere)."""
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["small"]
    W = I.make_weights(shape)
    model = P.SRM(shape, W, device=DEV)
    B, n_max = 512, 24
    rng = np.random.default_rng(5)
    lengths = rng.integers(1, n_max + 1, size=B).astype(np.int32)
    lengths[:3] = (n_max, 1, 2)
    toks = _ragged_batch(shape, [int(v) for v in lengths], seed=31)
    lens_dev = torch.from_numpy(lengths).to(DEV)
    g = P.Sampling("greedy")
    res = []
    for samples in (B, 64):
        st = model.new_state(B)
        ws = model.new_workspace(B, n_max, prefill_samples=samples)
        tok, lg = model.prefill_ragged(st, torch.from_numpy(toks).to(DEV), lens_dev, g, ws, want_logits=True)
        res.append((tok.cpu().numpy(), lg.cpu().numpy(), st.cache().cpu().numpy()))
        assert st.status() == 0
    # (eight bf16 layers: a last-bit difference in x now and then flips the bf16 rounding of an activation)
    assert rel_err_rows(res[0][1], res[1][1]) < 2e-2
    assert rel_err_rows(res[0][2], res[1][2]) < 2e-2
    assert (res[0][0] == res[1][0]).mean() > 0.9


def test_resume_of_a_ragged_state_from_a_copied_buffer():
    """generate(2k) == generate(k), copy the state buffer into a fresh state, adopt its positions, generate(k)."""
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["small"]
    model = P.SRM(shape, I.make_weights(shape), device=DEV)
    lengths = [20, 3, 11, 20]
    B, n_max, k = 4, 20, 5
    toks = torch.from_numpy(_ragged_batch(shape, lengths, seed=37)).to(DEV)
    lens_dev = torch.tensor(lengths, dtype=torch.int32, device=DEV)
    g = P.Sampling("topk", 50, 0.8, seed=3, sample_idx_base=40)
    ws = model.new_workspace(B, n_max, prefill_samples=B)
    a = model.new_state(B)
    model.prefill_ragged(a, toks, lens_dev, g, ws)
    full = model.generate(a, 2 * k, 1, g, ws).clone()
    b = model.new_state(B)
    model.prefill_ragged(b, toks, lens_dev, g, ws)
    first = model.generate(b, k, 1, g, ws).clone()
    c = model.new_state(B)
    assert not c.ragged and b.ragged
    c.buf.copy_(b.buf)
    c.adopt_positions(b.pos)
    assert c.ragged and c.pos == n_max + k
    rest = model.generate(c, k, k + 1, g, ws)
    assert torch.equal(full, torch.cat([first, rest], 1))
    assert torch.equal(a.cache(), c.cache()) and a.status() == 0 and c.status() == 0


def test_captured_step_is_not_reused_across_a_change_of_position_mode():
    """srm_generate keeps the captured step for as long as state, workspace, sampling and output buffer stay
    the same. Whether the samples share one position or keep their own is part of what was captured (the
    kernels take the position vector or not), so a state that is reset and prefilled the other way on the SAME
    buffers must get a new capture: both orders give exactly the tokens and cache of the launch-by-launch loop."""
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["small"]
    W = I.make_weights(shape)
    lengths = [24, 9, 17, 24, 3, 12]
    B, n = len(lengths), max(lengths)
    toks = torch.from_numpy(_ragged_batch(shape, lengths, seed=23)).to(DEV)
    lens = torch.tensor(lengths, dtype=torch.int32, device=DEV)
    g = P.Sampling("greedy")
    for order in (("plain", "ragged", "plain"), ("ragged", "plain")):
        res = {}
        for flags in (P.FLAG_NO_GRAPH, P.FLAG_GRAPH):
            model = P.SRM(shape, W, device=DEV, flags=flags)
            st = model.new_state(B)
            ws = model.new_workspace(B, n, prefill_samples=B)
            out = torch.full((B, 6), -1, dtype=torch.int32, device=DEV)
            got = []
            for mode in order:
                st.reset()
                if mode == "plain":
                    first = model.prefill(st, toks, g, ws)
                else:
                    first = model.prefill_ragged(st, toks, lens, g, ws)
                model.generate(st, 6, 1, g, ws, out=out)
                got.append((first.clone(), out.clone(), st.cache().clone()))
                assert st.ragged == (mode == "ragged")
            assert st.status() == 0
            res[flags] = got
        for a_, b_ in zip(res[P.FLAG_NO_GRAPH], res[P.FLAG_GRAPH]):
            for x_, y_ in zip(a_, b_):
                assert torch.equal(x_, y_)
        # the two modes really differ (shorter samples stand at other positions)
        assert not torch.equal(res[P.FLAG_GRAPH][0][1], res[P.FLAG_GRAPH][1][1])
