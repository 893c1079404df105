"""End-to-end parity of the CUDA path (through the C ABI) with the CPU oracle on the benchmark
configurations: logits and cache within tolerance, token ids bit-exact under the margin rule,
prefill (sequence-parallel) == decode (recurrent) on the device, batch invariance, resume."""
import numpy as np
import pytest
import torch

import srm_inputs as I
from helpers import oracle_for, rel_err_rows, top2_margin

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = {"fp32": 1e-4, "bf16": 3e-2}       # max relative error per row (logits, cache)
MARGIN = 1e-2                            # tokens must agree where the oracle's top-2 gap exceeds this


def _build(name, **kw):
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS[name]
    W = I.make_weights(shape)
    return shape, W, P.SRM(shape, W, device=DEV, **kw)


def _teacher_forced(shape, W, model, prompts, gen, sampling=None, sample_idx=None, check_state=True):
    """Prefill + `gen` selections. The oracle free-runs; the device consumes the ORACLE's tokens
    (teacher forcing), so one early disagreement cannot cascade. Returns statistics."""
    import paper_2605_08696_b200 as P
    orc = oracle_for(shape, W)
    B, n = prompts.shape
    samp_o = sampling or {"mode": "greedy"}
    sidx = np.arange(B) if sample_idx is None else sample_idx
    toks_o, logits_o, state_o = orc.generate(prompts, gen, samp_o, sample_idx=sidx)

    samp = P.Sampling("greedy") if samp_o["mode"] == "greedy" else \
        P.Sampling("topk", samp_o["top_k"], samp_o["temperature"], samp_o["seed"], int(sidx[0]))
    if samp_o["mode"] != "greedy":
        assert np.array_equal(sidx, sidx[0] + np.arange(B))
    st = model.new_state(B)
    ws = model.new_workspace(B, n, prefill_samples=B)
    tol = TOL[shape.dtype]
    first, lg = model.prefill(st, torch.from_numpy(prompts).to(DEV), samp, ws, want_logits=True)
    worst, mism, exempt, checked = 0.0, 0, 0, 0
    tok_g = first.cpu().numpy()
    for k in range(gen):
        lg_np = lg.cpu().numpy()
        worst = max(worst, rel_err_rows(lg_np, logits_o[k]))
        if samp_o["mode"] == "greedy":
            # Both of the top two logits can move by the row's device error eps, so a decision is only
            # determined when the oracle's margin exceeds 2 eps. In fp32 mode eps ~ 1e-6 and the rule is the
            # plain 1e-2 margin; in bf16 mode eps (bounded by the logit tolerance asserted below) reaches
            # ~1e-2 on the 16- and 24-layer models, and the guard keeps a 0.0101 margin from counting.
            eps_row = np.max(np.abs(lg_np - logits_o[k]), axis=-1)
            strict = top2_margin(logits_o[k]) > np.maximum(MARGIN, 2.0 * eps_row)
            checked += int(strict.sum())
            mism += int(np.sum(tok_g[strict] != toks_o[strict, k]))
            exempt += int(np.sum(~strict))
        else:
            # (a) in situ, bit-exact: the oracle's sampler run on the DEVICE's fp32 logits must pick
            #     the device's token (same Philox key, sample index and step), except where u*total
            #     lies within 1e-6*total of a CDF edge (fp32 vs fp64 cumulative sums);
            # (b) against the free-running oracle: ids must agree wherever the oracle's decision is
            #     stable under the measured logit error eps of that row: the k-th/(k+1)-th gap
            #     exceeds 2 eps and u is farther than 2(exp(2 eps/T) - 1) from every CDF edge.
            from oracle import srm_oracle as O
            K, T = samp_o["top_k"], samp_o["temperature"]
            t_dev, det_dev = O.select_topk(lg_np, K, T, samp_o["seed"], sidx, k, return_detail=True)
            _, det_o = O.select_topk(logits_o[k], K, T, samp_o["seed"], sidx, k, return_detail=True)
            for b in range(B):
                if tok_g[b] != t_dev[b]:
                    c, thr = det_dev[b]["cdf"], det_dev[b]["thr"]
                    assert np.min(np.abs(c - thr)) < 1e-6 * c[-1], (k, b, tok_g[b], t_dev[b])
                order = O.topk_order(logits_o[k][b], K + 1)
                eps = np.max(np.abs(lg_np[b] - logits_o[k][b]))
                gap = logits_o[k][b][order[K - 1]] - logits_o[k][b][order[K]]
                c = det_o[b]["cdf"] / det_o[b]["cdf"][-1]
                stable = gap > 2 * eps and np.min(np.abs(c - det_o[b]["u"])) > 2 * (np.exp(2 * eps / T) - 1)
                if stable:
                    checked += 1
                    mism += int(tok_g[b] != toks_o[b, k])
                else:
                    exempt += 1
        if k + 1 < gen:
            tok_in = torch.from_numpy(toks_o[:, k].copy()).to(DEV)
            tok_dev, lg = model.decode_step(st, tok_in, samp, k + 1, ws, want_logits=True)
            tok_g = tok_dev.cpu().numpy()
    assert st.status() == 0
    assert st.pos == n + gen - 1
    if check_state:
        # the oracle's final state corresponds to the same consumed tokens
        cache = st.cache().cpu().numpy()
        assert rel_err_rows(cache, state_o) < tol
    assert worst < tol, f"logits rel err {worst}"
    return dict(worst=worst, mismatches=mism, checked=checked, exempt=exempt, tokens=toks_o)


def test_tiny_config_nucleus_sampling_follows_the_oracle_sampler_step_by_step():
    """Free-running generation with top-p 0.9 at temperature 0.7 (the paper's rollout sampler) on the tiny
    fp32 model: at every step the oracle's nucleus sampler, run on the logits the device produced, with the
    same Philox key, sample index and step, draws the device's token (decisions within rounding of flipping
    excepted); replicas of one prompt draw different continuations."""
    import paper_2605_08696_b200 as P
    from oracle import srm_oracle as O
    from helpers import topp_is_strict
    shape, W, model = _build("tiny")
    prompts = np.repeat(I.make_prompts("tiny")[:2], 8, axis=0)           # 2 prompts x 8 replicas
    B, n = prompts.shape
    p, T, seed, base = 0.9, 0.7, 99, 500
    samp = P.Sampling("topp", temperature=T, seed=seed, sample_idx_base=base, top_p=p)
    st = model.new_state(B)
    ws = model.new_workspace(B, n, prefill_samples=B)
    tok, lg = model.prefill(st, torch.from_numpy(prompts).to(DEV), samp, ws, want_logits=True)
    checked, seqs = 0, [tok.cpu().numpy().copy()]
    for k in range(20):
        lg_np, tok_np = lg.cpu().numpy(), tok.cpu().numpy()
        want, det = O.select_topp(lg_np, np.float32(p), T, seed, base + np.arange(B), k, return_detail=True)
        for b in range(B):
            if topp_is_strict(lg_np[b], float(np.float32(p)), T, det[b]):
                assert tok_np[b] == want[b], (k, b)
                checked += 1
        tok, lg = model.decode_step(st, None, samp, k + 1, ws, want_logits=True)
        seqs.append(tok.cpu().numpy().copy())
    assert checked > 0.9 * 20 * B
    seqs = np.stack(seqs, 1)
    assert len({tuple(r) for r in seqs[:8]}) > 4 and st.status() == 0


def test_decode_with_and_without_split_k_down_projection_agree():
    """The decode step shares the K dimension of the down projection out between CTA pairs where that is the
    faster kernel (the rollout model at 8192 rows: 192 tiles of 96 k-blocks for 74 pairs).
    Same products, another order of fp32 additions in x; through 16 bf16 layers a last-bit difference in x now
    and then flips the bf16 rounding of an activation, so the two runs differ by what bf16 inputs allow (the
    kernel-level test shows 1e-5 for one projection): both stay inside the bf16 tolerance of each other."""
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["rl"]
    W = I.make_weights(shape)
    B, n = 8192, 4
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=3)).to(DEV)
    res = []
    for flags in (0, P.FLAG_NO_SPLITK):
        model = P.SRM(shape, W, device=DEV, flags=flags)
        st = model.new_state(B)
        ws = model.new_workspace(B, n, prefill_samples=B)
        tok = model.prefill(st, prompts, P.Sampling("greedy"), ws)
        for k in range(2):
            tok, lg = model.decode_step(st, tok, P.Sampling("greedy"), k + 1, ws, want_logits=True)
        res.append((lg[:64].cpu().numpy(), st.cache()[:, :64].cpu().numpy(), st.status()))
    assert res[0][2] == 0 and res[1][2] == 0
    assert not np.array_equal(res[0][0], res[1][0])          # (the split kernel did run: other order of additions)
    assert rel_err_rows(res[0][0], res[1][0]) < 2e-2
    assert rel_err_rows(res[0][1], res[1][1]) < 2e-2


def test_tiny_config_full_parity_fp32():
    """Config 'tiny': 4 prompts x 8 tokens, greedy 24 tokens, fp32, tolerance 1e-4; every token
    with margin > 1e-2 bit-exact; also free-running generation equals the oracle's tokens."""
    import paper_2605_08696_b200 as P
    shape, W, model = _build("tiny")
    prompts = I.make_prompts("tiny")
    r = _teacher_forced(shape, W, model, prompts, 24)
    assert r["mismatches"] == 0 and r["checked"] > 0
    # free-running: prefill, then srm_generate for the remaining 23 tokens
    st = model.new_state(4)
    ws = model.new_workspace(4, 8, prefill_samples=4)
    first = model.prefill(st, torch.from_numpy(prompts).to(DEV), P.Sampling("greedy"), ws)
    rest = model.generate(st, 23, 1, P.Sampling("greedy"), ws)
    got = torch.cat([first[:, None], rest], 1).cpu().numpy()
    orc = oracle_for(shape, W)
    toks_o, logits_o, _ = orc.generate(prompts, 24)
    safe = np.cumprod(top2_margin(logits_o).T > MARGIN, axis=1).astype(bool)   # up to first thin margin
    assert np.array_equal(got[safe], toks_o[safe])
    assert st.pos == 31 and st.status() == 0


def test_tiny_parallel_form_on_full_sequences_equals_recurrent_on_device():
    """Prefill (sequence-parallel form) over the full 32-token sequences gives the cache and last
    logits that 32 recurrent steps give."""
    import paper_2605_08696_b200 as P
    shape, W, model = _build("tiny")
    full = I.uniform_prompts(4, 32, shape.vocab, seed=5)
    ws = model.new_workspace(4, 32, prefill_samples=4)
    g = P.Sampling("greedy")
    st_p = model.new_state(4)
    _, lg_p = model.prefill(st_p, torch.from_numpy(full).to(DEV), g, ws, want_logits=True)
    st_r = model.new_state(4)
    for t in range(32):
        _, lg_r = model.decode_step(st_r, torch.from_numpy(full[:, t].copy()).to(DEV), g, 0, ws, want_logits=True)
    assert rel_err_rows(lg_p.cpu().numpy(), lg_r.cpu().numpy()) < 1e-5
    assert rel_err_rows(st_p.cache().cpu().numpy(), st_r.cache().cpu().numpy()) < 1e-5
    orc = oracle_for(shape, W)
    lo, so = orc.forward_parallel(full)
    assert rel_err_rows(lg_p.cpu().numpy(), lo[:, -1]) < 1e-4
    assert rel_err_rows(st_p.cache().cpu().numpy(), so) < 1e-4
    with pytest.raises(P.SRMError):                 # position 32 does not exist (n_ctx = 32)
        model.decode_step(st_r, None, g, 0, ws)


def test_small_config_bf16_parity_subset():
    """Config 'small' (L8 d512 V8000 bf16): 16 of the 256 prompts, prefill 128, 24 decode steps."""
    shape, W, model = _build("small")
    prompts = I.make_prompts("small")[:16]
    r = _teacher_forced(shape, W, model, prompts, 25)
    assert r["mismatches"] == 0 and r["checked"] > 0.5 * 16 * 25


def test_small_config_bf16_state_dtype_parity():
    shape, W, model = _build("small", state_dtype="bf16")
    prompts = I.make_prompts("small")[:8]
    r = _teacher_forced(shape, W, model, prompts, 9)
    assert r["mismatches"] == 0


def test_small_config_batch_invariance_and_chunking():
    """Row b's tokens do not depend on the batch it is in, nor on how the batch is split into
    workspace-sized passes: B=256 in one pass == B=256 in passes of 48 == B=16 alone, bit for bit."""
    import paper_2605_08696_b200 as P
    shape, W, model = _build("small")
    prompts = I.make_prompts("small")
    g = P.Sampling("greedy")
    outs = []
    for B, chunk in [(256, 256), (256, 48), (16, 16)]:
        st = model.new_state(B)
        ws = model.new_workspace(chunk, 128, prefill_samples=max(1, chunk // 8))
        first = model.prefill(st, torch.from_numpy(prompts[:B]).to(DEV), g, ws)
        rest = model.generate(st, 12, 1, g, ws)
        outs.append(torch.cat([first[:, None], rest], 1).cpu().numpy())
        assert st.status() == 0
    assert np.array_equal(outs[0], outs[1])
    assert np.array_equal(outs[0][:16], outs[2])


def test_fused_greedy_head_equals_logits_then_selection_on_device():
    """srm_generate / srm_prefill select inside the LM-head epilogue when no logits are requested; asking
    for the logits takes the LM head + selection-kernel route. Free-running, both must emit the same ids."""
    import paper_2605_08696_b200 as P
    shape, W, model = _build("small")
    B, n, gen = 70, 128, 10
    prompts = torch.from_numpy(I.make_prompts("small")[:B]).to(DEV)
    g = P.Sampling("greedy")
    ws = model.new_workspace(B, n, prefill_samples=B)
    st_a, st_b = model.new_state(B), model.new_state(B)
    first_a = model.prefill(st_a, prompts, g, ws)                        # fused
    rest_a = model.generate(st_a, gen, 1, g, ws)                         # fused
    first_b, _ = model.prefill(st_b, prompts, g, ws, want_logits=True)   # logits + selection kernel
    toks_b, tok = [first_b], first_b
    for k in range(gen):
        tok, _ = model.decode_step(st_b, tok, g, k + 1, ws, want_logits=True)
        toks_b.append(tok.clone())
    assert torch.equal(torch.cat([first_a[:, None], rest_a], 1), torch.stack(toks_b, 1))
    assert st_a.status() == 0 and st_b.status() == 0


@pytest.mark.parametrize("mode", ["greedy", "topk", "topp"])
def test_replicated_prefill_equals_prefill_of_the_replicated_prompts(mode):
    """srm_prefill_replicated (each distinct prompt run once, cache copied to its replicas, one selection per
    replica) leaves, bit for bit, what srm_prefill on the replicated token matrix leaves: cache, first tokens,
    and the tokens of the following decode steps. Several passes (small workspace) included."""
    import paper_2605_08696_b200 as P
    shape, W, model = _build("small")
    n_prompts, replicas, n = 5, 7, 40
    B = n_prompts * replicas
    base = torch.from_numpy(I.uniform_prompts(n_prompts, n, shape.vocab, seed=31)).to(DEV)
    full = base.repeat_interleave(replicas, dim=0).contiguous()
    samp = {"greedy": P.Sampling("greedy"), "topk": P.Sampling("topk", 50, 0.8, seed=77, sample_idx_base=1000),
            "topp": P.Sampling("topp", temperature=0.7, seed=77, sample_idx_base=1000, top_p=0.9)}[mode]
    ws = model.new_workspace(B, n, prefill_samples=B + 8)
    st_a, st_b, st_c = model.new_state(B), model.new_state(B), model.new_state(B)
    first_a = model.prefill(st_a, full, samp, ws)
    first_b, lg_b = model.prefill_replicated(st_b, base, replicas, samp, ws, want_logits=True)
    ws_small = model.new_workspace(4, n, prefill_samples=3)                  # two prompts per pass at most
    first_c = model.prefill_replicated(st_c, base, replicas, samp, ws_small)
    assert torch.equal(first_a, first_b) and torch.equal(first_a, first_c)
    assert torch.equal(st_a.cache(), st_b.cache()) and torch.equal(st_a.cache(), st_c.cache())
    assert lg_b.shape == (n_prompts, shape.vocab)
    if mode != "greedy":
        assert len(set(first_a[:replicas].tolist())) > 1                     # replicas of one prompt draw differently
    else:
        assert len(set(first_a[:replicas].tolist())) == 1
    for k in range(1, 4):
        ta = model.decode_step(st_a, None, samp, k, ws)
        tb = model.decode_step(st_b, None, samp, k, ws)
        assert torch.equal(ta, tb)
    assert st_a.status() == 0 and st_b.status() == 0 and st_c.status() == 0 and st_b.pos == n + 3


@pytest.mark.parametrize("mode", ["greedy", "topk", "topp"])
def test_generate_by_graph_replay_equals_launch_by_launch(mode):
    """srm_generate replaying one captured step (position, Philox step and store column in device-side
    counters) emits exactly the tokens and leaves exactly the cache of the launch-by-launch loop; a second call
    on the same buffers reuses the graph and continues correctly; a new output buffer re-captures."""
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["small"]
    W = I.make_weights(shape)
    m_loop = P.SRM(shape, W, device=DEV, flags=P.FLAG_NO_GRAPH)
    m_graph = P.SRM(shape, W, device=DEV, flags=P.FLAG_GRAPH)
    B, n = 48, 32
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=41)).to(DEV)
    samp = {"greedy": P.Sampling("greedy"), "topk": P.Sampling("topk", 50, 0.8, seed=5, sample_idx_base=7),
            "topp": P.Sampling("topp", temperature=0.7, seed=5, sample_idx_base=7, top_p=0.9)}[mode]
    outs = []
    for model in (m_loop, m_graph):
        st = model.new_state(B)
        ws = model.new_workspace(20, n, prefill_samples=B)        # 20-row passes: three chunks per step
        first = model.prefill(st, prompts, samp, ws)
        out = torch.full((B, 16), -1, dtype=torch.int32, device=DEV)
        model.generate(st, 9, 1, samp, ws, out=out[:, :9])
        assert st.pos == n + 9
        model.generate(st, 7, 10, samp, ws, out=out[:, 9:])
        out2 = model.generate(st, 5, 17, samp, ws)                # fresh output buffer
        assert st.pos == n + 21 and st.status() == 0
        outs.append((first.clone(), out.clone(), out2.clone(), st.cache().clone()))
    for a_, b_ in zip(outs[0], outs[1]):
        assert torch.equal(a_, b_)
    assert (outs[1][1] >= 0).all()


def test_resume_from_exported_cache():
    """generate(2k) == generate(k), copy the state buffer, generate(k) on the copy."""
    import paper_2605_08696_b200 as P
    shape, W, model = _build("small")
    prompts = I.make_prompts("small")[:32]
    g = P.Sampling("greedy")
    ws = model.new_workspace(32, 128, prefill_samples=8)
    st = model.new_state(32)
    model.prefill(st, torch.from_numpy(prompts).to(DEV), g, ws)
    a = model.generate(st, 10, 1, g, ws).cpu().numpy()
    st2 = model.new_state(32)
    model.prefill(st2, torch.from_numpy(prompts).to(DEV), g, ws)
    b1 = model.generate(st2, 5, 1, g, ws).cpu().numpy()
    st3 = model.new_state(32)
    st3.buf.copy_(st2.buf)
    st3.pos = st2.pos
    b2 = model.generate(st3, 5, 6, g, ws).cpu().numpy()
    assert np.array_equal(a, np.concatenate([b1, b2], 1))


def test_mid_config_bf16_parity_subset():
    """Config 'mid' (L16 d1024 V32000 bf16, Zipf prompts of 256): 8 samples, 6 decode steps."""
    shape, W, model = _build("mid")
    prompts = I.make_prompts("mid", batch=8)
    r = _teacher_forced(shape, W, model, prompts, 7)
    assert r["mismatches"] == 0 and r["checked"] > 0


def test_rl_config_topk_philox_parity_subset():
    """Config 'rl' (L24 d1536 V32000 bf16): one replica of 8 of the 16 distinct prompts,
    consecutive Philox sample indices, top-k 50, T 0.8."""
    shape, W, model = _build("rl")
    prompts = I.make_prompts("rl", batch=16 * 8)[::16][:8]          # 8 distinct prompts
    samp = dict(mode="topk", top_k=50, temperature=0.8, seed=3)
    r = _teacher_forced(shape, W, model, prompts, 5, sampling=samp, sample_idx=np.arange(8) + 7)
    # Random-init logits are nearly flat, so membership of the top-50 set is rarely stable under
    # the bf16 logit error: most free-running comparisons are exempt by rule (b) and the in-situ
    # check (a), asserted inside for all 8 x 5 decisions, is the bit-exact one.
    assert r["mismatches"] == 0
    assert r["checked"] + r["exempt"] == 8 * 5


def test_host_buffer_step_matches_device_step():
    import paper_2605_08696_b200 as P
    shape, W, model = _build("small")
    prompts = I.make_prompts("small")[:8]
    g = P.Sampling("greedy")
    ws = model.new_workspace(8, 128, prefill_samples=8)
    st = model.new_state(8); st2 = model.new_state(8)
    f1 = model.prefill(st, torch.from_numpy(prompts).to(DEV), g, ws)
    model.prefill(st2, torch.from_numpy(prompts).to(DEV), g, ws)
    d_out = model.decode_step(st, f1, g, 1, ws).cpu()
    h_in = f1.cpu().pin_memory(); h_out = torch.empty(8, dtype=torch.int32).pin_memory()
    model.decode_step_host(st2, h_in, g, 1, h_out, ws)
    torch.cuda.synchronize()
    assert torch.equal(d_out, h_out)
