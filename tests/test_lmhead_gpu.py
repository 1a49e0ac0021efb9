"""GPU parity of the output layer's gradient (``sd_lmhead_grad``: dW = g^T X on the tensor cores)
against the CPU oracle, through the C ABI.

Bar: both operands are bf16, every product of two of them is exact in fp32, and the accumulation
runs in fp32 over R terms; so an entry may be off by the rounding of that accumulation,
|gpu - ref| <= 2e-5 * sum_r |g[r,v] x[r,j]| (the bound written here is R * 2^-24 with R <= 2048,
doubled), whatever cancels in the sum itself.
"""
import numpy as np
import pytest
import torch

from oracle import sd_oracle
from paper_2603_12617_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-5


@pytest.fixture(scope="module")
def binding():
    import __graft_entry__ as entry
    entry.build()
    from paper_2603_12617_b200 import binding as b
    return b


def operands(R, V, d, seed):
    """Gradient-like g (most entries tiny, a few large, rows summing to about zero) and N(0,1) hidden
    states, both rounded to bf16."""
    rng = np.random.default_rng(seed)
    g = rng.normal(0, 1e-3, (R, V)).astype(np.float32)
    hot = rng.integers(0, V, (R, 3))
    g[np.arange(R)[:, None], hot] += rng.normal(0, 0.3, (R, 3)).astype(np.float32)
    X = rng.normal(0, 1, (R, d)).astype(np.float32)
    return synth.f32_to_bf16_bits(g), synth.f32_to_bf16_bits(X)


def dev_bf16(bits):
    return torch.from_numpy(bits).cuda().view(torch.bfloat16)


def abs_sum(gb, Xb, vs, js):
    g = np.abs(synth.bf16_bits_to_f32(gb).astype(np.float64))
    X = np.abs(synth.bf16_bits_to_f32(Xb).astype(np.float64))
    return np.einsum("re,re->e", g[:, vs], X[:, js])


@pytest.mark.parametrize("R,V,d", [(64, 128, 256), (70, 264, 80), (1, 8, 8), (200, 1000, 512), (129, 128 * 3 + 8, 256 + 64)])
def test_small_shapes_every_entry(binding, R, V, d):
    """Whole tiles and ragged ones in every dimension (positions not a multiple of 64, vocabulary not a
    multiple of 128, features not a multiple of 256)."""
    gb, Xb = operands(R, V, d, seed=R * 1000 + V)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    guard = torch.full((V * d + 128,), -7.0, dtype=torch.float32, device="cuda")
    out = guard[64:64 + V * d].view(V, d)
    binding.sd_lmhead_grad(dev_bf16(gb), dev_bf16(Xb), out=out, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert (guard[:64] == -7).all() and (guard[-64:] == -7).all(), "written outside dW"
    ref = sd_oracle.lmhead_grad(gb, Xb)
    vs, js = np.meshgrid(np.arange(V), np.arange(d), indexing="ij")
    bound = TOL * abs_sum(gb, Xb, vs.ravel(), js.ravel()).reshape(V, d) + 1e-30
    err = np.abs(out.cpu().numpy().astype(np.float64) - ref)
    assert (err <= bound).all(), f"worst ratio {np.max(err / bound):.3g} at {np.unravel_index(np.argmax(err / bound), err.shape)}"
    assert binding.sd_launch_info()["path"] == 5


def test_full_size_sampled(binding):
    """The shape the benchmark times (R = 256*6 positions, V = 128256, d = 4096): entries sampled over
    the whole of dW, including the corners of tiles, each computed by the oracle on its own."""
    R, V, d = 1536, 128256, 4096
    gb, Xb = operands(R, V, d, seed=7)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = binding.sd_lmhead_grad(dev_bf16(gb), dev_bf16(Xb), status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    rng = np.random.default_rng(8)
    vs = np.concatenate([rng.integers(0, V, 3000), [0, 127, 128, V - 1, V - 128, 64, 63, 65535, 65536]])
    js = np.concatenate([rng.integers(0, d, 3000), [0, 255, 256, d - 1, d - 256, 4095, 31, 32, 2048]])
    ref = sd_oracle.lmhead_grad(gb, Xb, vs, js)
    got = out[torch.from_numpy(vs).cuda(), torch.from_numpy(js).cuda()].cpu().numpy().astype(np.float64)
    bound = TOL * abs_sum(gb, Xb, vs, js) + 1e-30
    err = np.abs(got - ref)
    assert (err <= bound).all(), f"worst ratio {np.max(err / bound):.3g}"
    # a property that holds for every entry: the columns of dW add up to X^T (sum over v of g[:,v])
    colsum = out.sum(dim=0, dtype=torch.float64).cpu().numpy()
    gsum = synth.bf16_bits_to_f32(gb).astype(np.float64).sum(axis=1)
    want = synth.bf16_bits_to_f32(Xb).astype(np.float64).T @ gsum
    scale = np.abs(synth.bf16_bits_to_f32(Xb).astype(np.float64)).T @ np.abs(synth.bf16_bits_to_f32(gb).astype(np.float64)).sum(axis=1)
    assert (np.abs(colsum - want) <= 1e-4 * scale + 1e-12).all()


def test_gradient_of_the_step_feeds_the_output_layer(binding):
    """The real chain: the feedback step's gradient (bf16) goes straight into sd_lmhead_grad."""
    cfg = synth.custom_config(B=5, k=3, V=4096 + 128, dtype="bf16", tau=0.9, index=77)
    inp = synth.make_inputs(cfg)
    T = torch.from_numpy(inp.target_logits).cuda().view(torch.bfloat16)
    D = torch.from_numpy(inp.draft_logits).cuda().view(torch.bfloat16)
    step = binding.sd_verify_feedback(T, D, torch.from_numpy(inp.draft_tokens).cuda(), torch.from_numpy(inp.uniforms).cuda(), inp.tau)
    rng = np.random.default_rng(9)
    Xb = synth.f32_to_bf16_bits(rng.normal(0, 1, (cfg.B * cfg.k, 320)).astype(np.float32))
    dW = binding.sd_lmhead_grad(step.grad_draft, dev_bf16(Xb))
    torch.cuda.synchronize()
    gb = step.grad_draft.view(torch.int16).cpu().numpy().view(np.uint16).reshape(cfg.B * cfg.k, cfg.V)
    ref = sd_oracle.lmhead_grad(gb, Xb)
    vs, js = np.meshgrid(np.arange(cfg.V), np.arange(320), indexing="ij")
    bound = TOL * abs_sum(gb, Xb, vs.ravel(), js.ravel()).reshape(cfg.V, 320) + 1e-30
    assert (np.abs(dW.cpu().numpy().astype(np.float64) - ref) <= bound).all()


def test_refusals(binding):
    g = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    X = torch.zeros((8, 16), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.SdVerifyError):          # V not a multiple of 8
        binding.sd_lmhead_grad(torch.zeros((8, 60), dtype=torch.bfloat16, device="cuda"), X)
    with pytest.raises(binding.SdVerifyError):          # d not a multiple of 8
        binding.sd_lmhead_grad(g, torch.zeros((8, 12), dtype=torch.bfloat16, device="cuda"))
    with pytest.raises(TypeError):
        binding.sd_lmhead_grad(g.float(), X)
    with pytest.raises(ValueError):
        binding.sd_lmhead_grad(g, torch.zeros((9, 16), dtype=torch.bfloat16, device="cuda"))
