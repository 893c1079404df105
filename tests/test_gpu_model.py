"""End-to-end parity of the CUDA path (through the C ABI) with the CPU oracle on the benchmark
configurations: logits and cache within tolerance, token ids bit-exact under the margin rule,
prefill (sequence-parallel) == decode (recurrent) on the device, batch invariance, resume."""
import numpy as np
import pytest
import torch

import srm_inputs as I
from helpers import oracle_for, rel_err_rows, top2_margin, weights_for
from parity import DEV, MARGIN, assert_greedy_coverage, teacher_forced

pytestmark = pytest.mark.gpu


def _build(name, **kw):
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS[name]
    W = weights_for(name)
    kw["flags"] = kw.get("flags", 0) | P.FLAG_NO_SMALL_BATCH      # these tests are about the kernel-per-operation path
    return shape, W, P.SRM(shape, W, device=DEV, **kw)


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
    W = weights_for("rl")
    B, n = 8192, 4
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=3)).to(DEV)
    res = []
    # (with the feed-forward block as two launches: the single-kernel block never splits K)
    for flags in (P.FLAG_NO_FUSED_FFN, P.FLAG_NO_FUSED_FFN | P.FLAG_NO_SPLITK):
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
    r = teacher_forced("tiny", shape, W, model, prompts, 24, run_to_ctx_end=True)
    assert r["guarded"] == 0 and r["plain_mismatches"] == 0          # fp32: the plain 1e-2 rule, no guard needed
    assert_greedy_coverage(r, 0.0)
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
    r = teacher_forced("small", shape, W, model, prompts, 25)
    assert_greedy_coverage(r, 0.02)


def test_small_config_bf16_state_dtype_parity():
    shape, W, model = _build("small", state_dtype="bf16")
    prompts = I.make_prompts("small")[:8]
    r = teacher_forced("small/bf16-cache", shape, W, model, prompts, 9)
    assert_greedy_coverage(r, 0.20)          # 72 decisions: ten guarded ones are already 15 %


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
    W = weights_for("small")
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
    r = teacher_forced("mid", shape, W, model, prompts, 7)
    assert_greedy_coverage(r, 0.10)


def test_rl_config_topk_philox_parity_subset():
    """Config 'rl' (L24 d1536 V32000 bf16): one replica of 8 of the 16 distinct prompts,
    consecutive Philox sample indices, top-k 50, T 0.8."""
    shape, W, model = _build("rl")
    prompts = I.make_prompts("rl", batch=16 * 8)[::16][:8]          # 8 distinct prompts
    samp = dict(mode="topk", top_k=50, temperature=0.8, seed=3)
    r = teacher_forced("rl", shape, W, model, prompts, 5, sampling=samp, sample_idx=np.arange(8) + 7)
    # Random-init logits are nearly flat, so membership of the top-50 set is rarely stable under the bf16 logit
    # error: few free-running comparisons are determined (rule (b)); the in-situ check (a), made for all 8 x 5
    # decisions, is the bit-exact one, and at most a few of them may sit on a CDF edge.
    assert r["in_situ_checked"] + r["in_situ_edge"] == 8 * 5 and r["in_situ_checked"] >= 0.9 * 8 * 5


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
