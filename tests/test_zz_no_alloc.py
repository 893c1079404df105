"""srm_decode_step_static: the decode step for callers that cannot allocate device memory (a plug-in
inside an application that reserved the whole GPU, a loop that must not take cudaMalloc's implicit
synchronisation). Its workspace is an array built into the library, so the call takes no workspace
argument. It must give what srm_decode_step gives with a caller-allocated workspace.

Collected last on purpose (file name): a run that stops at the first failure has then already
executed every other test. The test needs no state left behind by other tests and leaves none that
matters: the built-in array is scratch, fully rewritten by every call.
"""
import numpy as np
import pytest
import torch

import srm_inputs as I
from helpers import rel_err_rows

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = {"fp32": 1e-4, "bf16": 3e-2}     # the tolerances of the model-level parity tests


BF16_SHAPE = I.SRMShape(n_layers=2, d_model=256, vocab=1000, n_ctx=32, dtype="bf16", seed=7)


@pytest.mark.parametrize("shape,B", [(I.CONFIGS["tiny"], 4), (BF16_SHAPE, 300), (BF16_SHAPE, 40)])     # 40: the single-kernel step
def test_static_scratch_step_matches_workspace_step_twice_in_a_row(shape, B):
    import paper_2605_08696_b200 as P
    from helpers import oracle_for
    W = I.make_weights(shape)
    model = P.SRM(shape, W, device=DEV)
    g = P.Sampling("greedy")
    n = 6
    prompts_np = I.uniform_prompts(B, n, shape.vocab, seed=11)
    prompts = torch.from_numpy(prompts_np).to(DEV)
    ws = model.new_workspace(B, n, prefill_samples=B)
    st_ref, st_new = model.new_state(B), model.new_state(B)
    first = model.prefill(st_ref, prompts, g, ws)
    model.prefill(st_new, prompts, g, ws)
    tok = first
    toks, logits = [first.cpu().numpy()], []
    for k in range(2):                                   # two calls in a row share the built-in array
        t_ref, lg_ref = model.decode_step(st_ref, tok, g, k + 1, ws, want_logits=True)
        t_new, lg_new = model.decode_step_static(st_new, tok, g, k + 1, want_logits=True)
        torch.cuda.synchronize()
        assert rel_err_rows(lg_new.cpu().numpy(), lg_ref.cpu().numpy()) < TOL[shape.dtype]
        assert torch.equal(t_new, t_ref)
        assert rel_err_rows(st_new.cache().cpu().numpy(), st_ref.cache().cpu().numpy()) < TOL[shape.dtype]
        # the two calls run the same kernels in the same order on the same inputs: not a bit may differ
        assert torch.equal(lg_new, lg_ref) and torch.equal(st_new.cache(), st_ref.cache())
        tok = t_ref
        toks.append(t_ref.cpu().numpy()); logits.append(lg_new.cpu().numpy())
    assert st_new.pos == st_ref.pos == n + 2
    assert st_new.status() == 0 and st_ref.status() == 0
    # and once against the CPU oracle fed the same tokens
    orc = oracle_for(shape, W)
    _, state = orc.forward_parallel(prompts_np)
    for k in range(2):
        lo, state = orc.decode_step(state, toks[k], n + k)
        assert rel_err_rows(logits[k], lo) < TOL[shape.dtype]


@pytest.mark.parametrize("mode", ["greedy_fused", "topk", "topp"])
def test_static_scratch_step_on_the_other_selection_paths(mode):
    """The paths that use the workspace differently from the logits-returning greedy step: selection fused into
    the LM head (its partial results live where the logits would), top-k and top-p on logits kept in the
    scratch array. Each must equal the workspace step exactly, two calls in a row."""
    import paper_2605_08696_b200 as P
    shape, B, n = BF16_SHAPE, 300, 5
    model = P.SRM(shape, I.make_weights(shape), device=DEV)
    samp = {"greedy_fused": P.Sampling("greedy"),
            "topk": P.Sampling("topk", 50, 0.8, seed=9, sample_idx_base=40),
            "topp": P.Sampling("topp", temperature=0.7, seed=9, sample_idx_base=40, top_p=0.9)}[mode]
    prompts = torch.from_numpy(I.uniform_prompts(B, n, shape.vocab, seed=12)).to(DEV)
    ws = model.new_workspace(B, n, prefill_samples=B)
    st_ref, st_new = model.new_state(B), model.new_state(B)
    model.prefill(st_ref, prompts, samp, ws)
    model.prefill(st_new, prompts, samp, ws)
    for k in range(2):
        t_ref = model.decode_step(st_ref, None, samp, k + 1, ws)
        t_new = model.decode_step_static(st_new, None, samp, k + 1)
        assert torch.equal(t_new, t_ref)
        assert torch.equal(st_new.cache(), st_ref.cache())
    assert st_new.status() == 0 and st_ref.status() == 0


def test_static_scratch_step_allocates_no_device_memory():
    """Free device memory, as the driver reports it, is the same before and after calls that pass preallocated
    outputs (the first call on a device may load kernels, so one call is made before the reading)."""
    import paper_2605_08696_b200 as P
    shape, B = BF16_SHAPE, 300
    model = P.SRM(shape, I.make_weights(shape), device=DEV)
    g = P.Sampling("greedy")
    st = model.new_state(B)
    st.pos = 3
    tok_in = torch.zeros(B, dtype=torch.int32, device=DEV)
    tok_out = torch.empty(B, dtype=torch.int32, device=DEV)
    model.decode_step_static(st, tok_in, g, 1, tok_out=tok_out)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    reserved0 = torch.cuda.memory_reserved()
    for k in range(3):
        model.decode_step_static(st, tok_in, g, 2 + k, tok_out=tok_out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0 and torch.cuda.memory_reserved() == reserved0
    assert st.status() == 0


def test_static_scratch_step_rejects_a_batch_that_does_not_fit():
    import paper_2605_08696_b200 as P
    shape = I.CONFIGS["tiny"]
    model = P.SRM(shape, I.make_weights(shape), device=DEV)
    B = 20000                                            # 20000 rows x 2.3 KB of workspace > 32 MiB
    assert model.workspace_bytes(B) > 32 << 20
    st = model.new_state(B)
    st.pos = 1
    with pytest.raises(P.SRMError) as e:
        model.decode_step_static(st, None, P.Sampling("greedy"), 1)
    assert e.value.code == -8
    assert "scratch" in str(e.value)
    assert st.pos == 1                                   # nothing was enqueued, nothing advanced
