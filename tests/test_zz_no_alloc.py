"""The entry point that allocates nothing (``sd_verify_feedback_static``).

Some callers of this library cannot allocate device memory while they run: a serving loop whose
memory was handed out once at start-up, a process held to a fixed footprint, a callback that must
not synchronise the device.  For them the library carries its scratch inside its own image.  This
file checks, through the C ABI, that the entry point gives the same answers as
``sd_verify_feedback_ex`` on two calls in a row (the second call finds the scratch as the first
one left it), and that a shape too large for the built-in scratch is refused on the host.

It is collected last on purpose, so that a run that stops at the first failure has already been
through every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2603_12617_b200 import synth

TOL = {"f32": 1e-5, "bf16": 2e-2}


@pytest.fixture(scope="module")
def binding():
    import __graft_entry__ as entry
    entry.build()
    from paper_2603_12617_b200 import binding as b
    return b


def test_oversized_shape_is_refused_on_the_host(binding):
    """No GPU needed: the size check comes before anything touches a device."""
    lib = binding._lib
    buf = (ctypes.c_float * 64)()
    p = ctypes.cast(buf, ctypes.c_void_p)
    B, k, V = 4096, 7, 131072
    assert lib.sd_workspace_bytes(B, k, V, 0) > binding.SD_STATIC_SCRATCH_BYTES
    rc = lib.sd_verify_feedback_static(p, p, p, p, 1.0, B, k, V, 0, p, p, p, p, None, None, None)
    assert rc == -4                                   # SD_ERR_WORKSPACE
    assert b"sd_verify_feedback_ex" in lib.sd_last_cuda_error()
    # argument errors are reported as by the other entry points
    assert lib.sd_verify_feedback_static(None, p, p, p, 1.0, 1, 1, 4, 0, p, p, p, p, None, None, None) == -1


def _outputs(binding, cfg, dev):
    dt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    return binding.StepOutputs(
        accept_len=torch.full((cfg.B,), -7, dtype=torch.int32, device=dev),
        tokens=torch.full((cfg.B, cfg.k + 1), -7, dtype=torch.int32, device=dev),
        loss=torch.full((cfg.B, cfg.k), -7.0, dtype=torch.float32, device=dev),
        grad_draft=torch.full((cfg.B, cfg.k, cfg.V), -7.0, dtype=dt, device=dev),
        acc_prob=torch.full((cfg.B, cfg.k), -7.0, dtype=torch.float32, device=dev),
        status=torch.full((cfg.B,), -7, dtype=torch.int32, device=dev))


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,B,k,V", [("f32", 6, 3, 20000), ("bf16", 5, 4, 50000), ("f32", 3, 2, 1001)])
def test_static_scratch_matches_caller_scratch_twice_in_a_row(binding, dtype, B, k, V):
    dev = torch.device("cuda", 0)
    tol = TOL[dtype]
    for call in range(2):
        # different inputs on the second call: whatever the first call left in the scratch must not matter
        cfg = synth.custom_config(B=B, k=k, V=V, dtype=dtype, tau=0.9, index=90 + call)
        inp = synth.make_inputs(cfg)
        T = torch.from_numpy(inp.target_logits).to(dev)
        D = torch.from_numpy(inp.draft_logits).to(dev)
        if dtype == "bf16":
            T, D = T.view(torch.bfloat16), D.view(torch.bfloat16)
        x = torch.from_numpy(inp.draft_tokens).to(dev)
        u = torch.from_numpy(inp.uniforms).to(dev)
        ref = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
        out = _outputs(binding, cfg, dev)
        assert binding.sd_workspace_bytes(B, k, V, binding._dtype_code(T)) <= binding.SD_STATIC_SCRATCH_BYTES
        binding.sd_verify_feedback_static(T, D, x, u, inp.tau, out=out)
        torch.cuda.synchronize()
        assert torch.equal(out.accept_len, ref.accept_len), f"call {call}: accept lengths differ"
        assert torch.equal(out.tokens, ref.tokens), f"call {call}: tokens differ"
        assert torch.equal(out.status, ref.status), f"call {call}: status differs"
        loss, rloss = out.loss.double().cpu().numpy(), ref.loss.double().cpu().numpy()
        assert (np.abs(loss - rloss) <= tol * np.abs(rloss) + 4e-7).all(), f"call {call}: loss differs"
        g, rg = out.grad_draft.double().cpu().numpy(), ref.grad_draft.double().cpu().numpy()
        bound = tol * np.abs(rg).max(axis=2, keepdims=True) + 1e-12
        assert (np.abs(g - rg) <= bound).all(), f"call {call}: gradient differs"
        assert torch.allclose(out.acc_prob, ref.acc_prob, rtol=0, atol=2e-5), f"call {call}: acc_prob differs"


@pytest.mark.gpu
def test_static_entry_point_allocates_nothing_and_survives_a_change_of_shape(binding):
    """What the entry point is for: once it has been called on a device, further calls leave the
    device's free memory exactly where it was -- also when the shape changes so that the words at
    the head of the built-in scratch move (batch sizes either side of 64) -- and still give the
    answers of sd_verify_feedback_ex."""
    dev = torch.device("cuda", 0)
    cases = []
    for i, (B, k, V) in enumerate([(5, 2, 4096), (130, 2, 4096), (5, 2, 4096), (64, 3, 2048), (65, 3, 2048)]):
        cfg = synth.custom_config(B=B, k=k, V=V, dtype="f32", tau=0.8, index=95 + i)
        inp = synth.make_inputs(cfg)
        T = torch.from_numpy(inp.target_logits).to(dev)
        D = torch.from_numpy(inp.draft_logits).to(dev)
        x = torch.from_numpy(inp.draft_tokens).to(dev)
        u = torch.from_numpy(inp.uniforms).to(dev)
        ref = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
        cases.append((cfg, inp, T, D, x, u, ref, _outputs(binding, cfg, dev)))
    cfg, inp, T, D, x, u, ref, out = cases[0]
    binding.sd_verify_feedback_static(T, D, x, u, inp.tau, out=out)      # the set-up call of this device
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info(dev)[0]
    for cfg, inp, T, D, x, u, ref, out in cases:
        binding.sd_verify_feedback_static(T, D, x, u, inp.tau, out=out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info(dev)[0] == free_before, "a call of the static entry point changed the free device memory"
    for cfg, inp, T, D, x, u, ref, out in cases:
        assert torch.equal(out.accept_len, ref.accept_len) and torch.equal(out.tokens, ref.tokens)
        assert torch.equal(out.status, ref.status)
        assert torch.equal(out.loss, ref.loss) and torch.equal(out.grad_draft, ref.grad_draft)
