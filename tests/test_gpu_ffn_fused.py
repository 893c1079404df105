"""The feed-forward block as one kernel (srm_k_ffn): up tiles and down tiles of one launch dealt to the CTA pairs by
a host-made plan, down tiles reading H as the up tiles complete. Every tile is still computed whole, by one pair, in
the same k-order, so the block must reproduce the two launches (up projection, then down projection) bit for bit, and
a decode step with it must equal a step without it in every logit and every cache value."""
import numpy as np
import pytest
import torch

import srm_inputs as I
from helpers import custom_shape, rel_err_rows

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _model(shape, **kw):
    import paper_2605_08696_b200 as P
    W = I.make_weights(shape, alpha_std=0.5, beta_std=0.5)
    return P.SRM(shape, W, device=DEV, **kw), W


def _ffn_inputs(m, shape, M, seed):
    rng = np.random.default_rng(seed)
    a = torch.from_numpy(rng.normal(size=(M, shape.d_model)).astype(np.float32)).to(DEV).to(torch.bfloat16)
    x0 = torch.from_numpy(rng.normal(size=(M, shape.d_model)).astype(np.float32)).to(DEV)
    return a, x0


@pytest.mark.parametrize("d,M", [(512, 1), (512, 100), (512, 256), (512, 700), (1024, 2048), (1024, 3000), (1024, 4096),
                                 (1536, 1300), (1024, 10240), (256, 16384)])
def test_fused_block_equals_the_two_launches_bit_for_bit(d, M):
    import paper_2605_08696_b200 as P
    shape = custom_shape(n_layers=2, d_model=d, vocab=512, n_ctx=16, dtype="bf16", seed=11)
    m, W = _model(shape)
    layer = 1
    F = 4 * d
    a, x0 = _ffn_inputs(m, shape, M, seed=d + M)
    W1, b1 = m.tensor(layer, P.binding.T_W1), m.tensor(layer, P.binding.T_B1)
    W2, b2 = m.tensor(layer, P.binding.T_W2), m.tensor(layer, P.binding.T_B2)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    # two launches
    H_ref = torch.zeros(M, F, dtype=torch.bfloat16, device=DEV)
    x_ref = x0.clone()
    m.k_gemm(P.EPI_BIAS_GELU, a, W1, b1, H_ref, status=status)
    m.k_gemm(P.EPI_BIAS_RESIDUAL, H_ref, W2, b2, x_ref, status=status)
    # one kernel, twice (the counters are cleared by the call; the scratch starts as garbage)
    nb = P.load_library().srm_k_ffn_ready_bytes(M, F)
    ready = torch.full((nb // 4,), 0x33333333, dtype=torch.int32, device=DEV)
    for _ in range(2):
        H = torch.full((M, F), float("nan"), dtype=torch.bfloat16, device=DEV)
        x = x0.clone()
        m.k_ffn(layer, a, H, x, ready=ready, status=status)
        torch.cuda.synchronize()
        assert status.item() == 0, f"device status {status.item()}"
        assert torch.equal(H.view(torch.int16), H_ref.view(torch.int16))
        assert torch.equal(x, x_ref)
    # and against the fp64 definition with the exact (erf) GELU, H rounded to bf16 as the kernel stores it
    if M <= 4096:
        from oracle import srm_oracle as O
        a64 = a.float().cpu().numpy().astype(np.float64)
        h = O.gelu_erf(a64 @ W1.float().cpu().numpy().astype(np.float64).T + b1.cpu().numpy().astype(np.float64))
        h = torch.from_numpy(h).to(torch.bfloat16).double().numpy()
        want = x0.cpu().numpy().astype(np.float64) + h @ W2.float().cpu().numpy().astype(np.float64).T + b2.cpu().numpy().astype(np.float64)
        assert rel_err_rows(x.cpu().numpy(), want) < 8e-3


def test_shapes_the_fused_block_does_not_take_are_refused():
    import paper_2605_08696_b200 as P
    shape = custom_shape(n_layers=1, d_model=320, vocab=512, n_ctx=16, dtype="bf16", seed=3)     # d not a multiple of 256
    m, _ = _model(shape)
    a, x = _ffn_inputs(m, shape, 64, seed=1)
    H = torch.zeros(64, 1280, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(P.SRMError) as e:
        m.k_ffn(0, a, H, x)
    assert e.value.code == P.ERR_UNSUPPORTED
    shape = custom_shape(n_layers=1, d_model=256, vocab=512, n_ctx=16, dtype="fp32", seed=3)     # fp32 model: SIMT path
    m, _ = _model(shape)
    with pytest.raises(P.SRMError) as e:
        m.k_ffn(0, torch.zeros(64, 256, device=DEV), torch.zeros(64, 1024, device=DEV), torch.zeros(64, 256, device=DEV))
    assert e.value.code == P.ERR_UNSUPPORTED


@pytest.mark.parametrize("B,d,head_proj,fused", [(2500, 1024, False, True), (3900, 512, True, True), (300, 512, False, False)])
def test_decode_steps_with_and_without_the_fused_block_are_equal(B, d, head_proj, fused):
    """Prefill and a few decode steps (logits requested, greedy) on two models over the same weights, one of them with
    SRM_FLAG_NO_FUSED_FFN: logits, tokens and cache must be equal, and the profile must show which path ran (the
    step takes the single kernel from two tiles per CTA pair; 300 rows of d = 512 are 20 tiles)."""
    import paper_2605_08696_b200 as P
    shape = custom_shape(n_layers=3, d_model=d, vocab=2048, n_ctx=24, dtype="bf16", seed=5, head_proj=head_proj)
    W = I.make_weights(shape, alpha_std=0.5, beta_std=0.5)
    base = P.FLAG_NO_SMALL_BATCH
    rng = np.random.default_rng(B)
    prompts = torch.from_numpy(rng.integers(0, shape.vocab, size=(B, 6)).astype(np.int32)).to(DEV)
    outs = []
    for flags in (base, base | P.FLAG_NO_FUSED_FFN):
        m = P.SRM(shape, W, device=DEV, flags=flags)
        st = m.new_state(B)
        ws = m.new_workspace(B, 6, prefill_samples=B)
        samp = P.Sampling("greedy")
        tok, _ = m.prefill(st, prompts, samp, ws, want_logits=True)
        m.profile(True)
        m.profile_reset()
        lgs = []
        for k in range(4):
            tok, lg = m.decode_step(st, tok, samp, k + 1, ws, want_logits=True)
            lgs.append(lg.clone())
        prof = m.profile_read()
        m.profile(False)
        assert st.status() == 0
        outs.append((torch.stack(lgs), tok.clone(), st.cache().clone(), prof))
    (lg_a, tok_a, S_a, prof_a), (lg_b, tok_b, S_b, prof_b) = outs
    if fused:
        assert prof_a["ffn"][0] == 4 * shape.n_layers and prof_a["gemm_up"][0] == 0
    else:
        assert prof_a["ffn"][0] == 0 and prof_a["gemm_up"][0] == 4 * shape.n_layers
    assert prof_b["ffn"][0] == 0 and prof_b["gemm_up"][0] == 4 * shape.n_layers
    assert torch.equal(lg_a, lg_b)
    assert torch.equal(tok_a, tok_b)
    assert torch.equal(S_a, S_b)


def test_captured_step_with_the_fused_block_equals_launch_by_launch():
    """srm_generate replaying a captured step whose feed-forward blocks are the single kernel (the work lists are
    part of the captured launch parameters, the counters are cleared by a captured memset) against the
    launch-by-launch loop: same tokens, same cache, also when the captured graph is replayed by a second call."""
    import paper_2605_08696_b200 as P
    shape = custom_shape(n_layers=3, d_model=512, vocab=2048, n_ctx=40, dtype="bf16", seed=8)
    W = I.make_weights(shape, alpha_std=0.5, beta_std=0.5)
    B, n = 3900, 4
    prompts = torch.from_numpy(np.random.default_rng(3).integers(0, shape.vocab, size=(B, n)).astype(np.int32)).to(DEV)
    samp = P.Sampling("topk", 20, 0.9, seed=4, sample_idx_base=11)
    outs = []
    for flags in (P.FLAG_NO_GRAPH, P.FLAG_GRAPH):
        m = P.SRM(shape, W, device=DEV, flags=flags)
        st = m.new_state(B)
        ws = m.new_workspace(B, n, prefill_samples=B)
        first = m.prefill(st, prompts, samp, ws)
        m.profile(True)
        m.profile_reset()
        a = m.generate(st, 6, 1, samp, ws)
        prof = m.profile_read()
        m.profile(False)
        b = m.generate(st, 5, 7, samp, ws, out=a[:, :5].clone())
        assert st.status() == 0 and st.pos == n + 11
        outs.append((first.clone(), a.clone(), b.clone(), st.cache().clone()))
        if flags == P.FLAG_NO_GRAPH:
            assert prof["ffn"][0] == 6 * shape.n_layers        # (launches inside a replayed graph are not bracketed)
    for x_, y_ in zip(outs[0], outs[1]):
        assert torch.equal(x_, y_)


def test_prefill_with_the_fused_block_in_slabs_equals_the_two_launches():
    """A prefill pass of more than 16384 rows runs its feed-forward blocks slab by slab through the single kernel (a
    whole slab, then a shorter one): logits of the last position, first tokens and the cache must equal the run with
    SRM_FLAG_NO_FUSED_FFN, and the decode step that follows must agree as well."""
    import paper_2605_08696_b200 as P
    shape = custom_shape(n_layers=2, d_model=1024, vocab=2048, n_ctx=320, dtype="bf16", seed=12)
    W = I.make_weights(shape, alpha_std=0.5, beta_std=0.5)
    B, n = 68, 300                                             # 20400 rows: one slab of 16384 and one of 4016
    prompts = torch.from_numpy(np.random.default_rng(5).integers(0, shape.vocab, size=(B, n)).astype(np.int32)).to(DEV)
    outs = []
    for flags in (0, P.FLAG_NO_FUSED_FFN):
        m = P.SRM(shape, W, device=DEV, flags=flags | P.FLAG_NO_SMALL_BATCH)
        st = m.new_state(B)
        ws = m.new_workspace(B, n, prefill_samples=B)
        m.profile(True)
        m.profile_reset()
        tok, lg = m.prefill(st, prompts, P.Sampling("greedy"), ws, want_logits=True)
        prof = m.profile_read()
        m.profile(False)
        tok2, lg2 = m.decode_step(st, tok, P.Sampling("greedy"), 1, ws, want_logits=True)
        assert st.status() == 0
        outs.append((lg.clone(), tok.clone(), lg2.clone(), st.cache().clone(), prof))
    assert outs[0][4]["ffn"][0] == 2 * shape.n_layers and outs[0][4]["gemm_up"][0] == 0
    assert outs[1][4]["ffn"][0] == 0 and outs[1][4]["gemm_up"][0] == shape.n_layers
    for a_, b_ in zip(outs[0][:4], outs[1][:4]):
        assert torch.equal(a_, b_)
