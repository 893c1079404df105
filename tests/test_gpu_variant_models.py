"""Models built from the two further token mixers of the Architecture section -- linearly combined heads (twice
the cache) and non-unitary kernels of size k (Eq. 11, k times the cache) -- through the same C-ABI calls as the
mixed-head model: srm_create with the mixer in the configuration, prefill, decode steps, generation. Parity
against the whole-model oracle that takes the variant (teacher-forced, logits at every step, the cache
[L, C, B, d] at the end), prefill == decode on the device, cache size accounting."""
import dataclasses

import numpy as np
import pytest
import torch

import srm_inputs as I
from helpers import oracle_for, rel_err_rows
from parity import DEV, assert_greedy_coverage, teacher_forced

pytestmark = pytest.mark.gpu
VARIANTS = [("combined", 1), ("kernel", 4), ("kernel", 8), ("kernel", 1), ("kernel", 13)]


def _build(base, mixer, k, **kw):
    import paper_2605_08696_b200 as P
    shape = dataclasses.replace(base, mixer=mixer, kernel_size=k)
    W = I.make_weights(shape)
    return shape, W, P.SRM(shape, W, device=DEV, **kw)


@pytest.mark.parametrize("mixer,k", VARIANTS)
def test_tiny_fp32_variant_model_full_parity(mixer, k):
    """fp32, d 64 (two channels per lane: the shifted reads cross lanes and vectors): 1e-4 on logits and cache over
    the whole context, tokens under the plain margin rule, the step past n_ctx refused."""
    shape, W, model = _build(I.CONFIGS["tiny"], mixer, k)
    r = teacher_forced("tiny", shape, W, model, I.make_prompts("tiny"), 24, run_to_ctx_end=True)
    assert r["guarded"] == 0 and r["plain_mismatches"] == 0
    assert_greedy_coverage(r, 0.0)
    C = {"combined": 2, "kernel": k}[mixer]
    st = model.new_state(3)
    assert model.planes == C and st.cache().shape == (shape.n_layers, C, 3, shape.d_model)


@pytest.mark.parametrize("mixer,k,state_dtype", [("combined", 1, "fp32"), ("kernel", 4, "fp32"), ("kernel", 8, "fp16"),
                                                 ("combined", 1, "fp16")])
def test_bf16_variant_model_parity_subset(mixer, k, state_dtype):
    """bf16 weights, d 512 (four vectors per lane) and d 1024 widths through the tensor-core GEMMs."""
    base = I.SRMShape(n_layers=4, d_model=512 if mixer == "kernel" else 1024, vocab=4096, n_ctx=96, dtype="bf16", seed=31)
    shape, W, model = _build(base, mixer, k, state_dtype=state_dtype)
    prompts = I.uniform_prompts(10, 40, shape.vocab, seed=6)
    r = teacher_forced("small", shape, W, model, prompts, 12)
    assert_greedy_coverage(r, 0.15)


@pytest.mark.parametrize("mixer,k", [("combined", 1), ("kernel", 8)])
def test_variant_prefill_equals_decode_on_device_and_replicated_prefill(mixer, k):
    """The sequence form (srm_prefill) leaves the cache and last logits that the recurrent steps leave, whatever the
    split into workspace passes; srm_prefill_replicated equals the prefill of the replicated prompts."""
    import paper_2605_08696_b200 as P
    base = I.SRMShape(n_layers=3, d_model=256, vocab=2048, n_ctx=48, dtype="bf16", seed=32)
    shape, W, model = _build(base, mixer, k)
    Pn, reps, n = 6, 5, 21
    basep = torch.from_numpy(I.uniform_prompts(Pn, n, shape.vocab, seed=7)).to(DEV)
    full = basep.repeat_interleave(reps, dim=0).contiguous()
    B = Pn * reps
    g = P.Sampling("greedy")
    ws = model.new_workspace(B, n, prefill_samples=B + 8)
    st_p, st_r, st_c, st_x = (model.new_state(B) for _ in range(4))
    _, lg_p = model.prefill(st_p, full, g, ws, want_logits=True)
    for t in range(n):
        _, lg_r = model.decode_step(st_r, full[:, t].contiguous(), g, 0, ws, want_logits=True)
    assert torch.equal(lg_p, lg_r) and torch.equal(st_p.cache(), st_r.cache())      # the same kernel, the same order
    ws_small = model.new_workspace(7, n, prefill_samples=4)
    _, lg_c = model.prefill(st_c, full, g, ws_small, want_logits=True)
    assert torch.equal(lg_c, lg_p) and torch.equal(st_c.cache(), st_p.cache())
    first_x = model.prefill_replicated(st_x, basep, reps, g, ws)
    assert torch.equal(st_x.cache(), st_p.cache())
    assert torch.equal(first_x, model.prefill(model.new_state(B), full, g, ws))
    a = model.generate(st_p, 6, 1, g, ws)
    b = model.generate(st_x, 6, 1, g, ws)
    assert torch.equal(a, b)
    for st in (st_p, st_r, st_c, st_x):
        assert st.status() == 0


def test_variant_configuration_limits():
    import paper_2605_08696_b200 as P
    tiny = I.CONFIGS["tiny"]
    for bad in (dataclasses.replace(tiny, mixer="kernel", kernel_size=17),
                dataclasses.replace(tiny, mixer="combined", head_proj=True)):
        with pytest.raises(P.SRMError):
            P.SRM(bad, I.make_weights(dataclasses.replace(bad, kernel_size=min(bad.kernel_size, 16))), device=DEV)
    with pytest.raises(P.SRMError):
        _build(tiny, "combined", 1, state_dtype="bf16")
    shape, W, model = _build(tiny, "combined", 1)
    st = model.new_state(4)
    ws = model.new_workspace(4, 8, prefill_samples=4)
    toks = torch.from_numpy(I.make_prompts("tiny")).to(DEV)
    lens = torch.tensor([8, 3, 5, 8], dtype=torch.int32, device=DEV)
    with pytest.raises(P.SRMError) as e:
        model.prefill_ragged(st, toks, lens, P.Sampling("greedy"), ws)
    assert e.value.code == P.ERR_UNSUPPORTED
