"""GPU parity of the error-position feedback (the signal OSD collects, Sec. 3.1) against the CPU
oracle, and against the full step of the same library.

Bars: verification exactly as in the full step (accept lengths and tokens bit-equal to
sd_verify_feedback on the same inputs; against the oracle bit-exact off the two threshold bands);
loss |gpu - ref| <= tol*|ref| + 4e-7; the gradient row max|gpu - ref| <= tol*max|ref| +
8*2^-24*max(p,q)/tau, tol = 1e-5 (fp32 logits) / 2e-2 (bf16 logits); a zero row where every draft
token was accepted.  Where the device's accept length differs from the oracle's (inside a band),
the row is compared with the oracle's row of the device's position.
"""
import numpy as np
import pytest
import torch

from oracle import sd_oracle
from paper_2603_12617_b200 import synth

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-2}
LOSS_FLOOR = 4e-7
GRAD_FLOOR = 8 * 2.0 ** -24


@pytest.fixture(scope="module")
def binding():
    import __graft_entry__ as entry
    entry.build()
    from paper_2603_12617_b200 import binding as b
    return b


def dev(a):
    t = torch.from_numpy(a).cuda()
    return t.view(torch.bfloat16) if a.dtype == np.uint16 else t


def f64(a):
    return (synth.bf16_bits_to_f32(a) if a.dtype == np.uint16 else a).astype(np.float64)


def pmax_of(z, tau):
    e = np.exp((z - z.max(axis=-1, keepdims=True)) / tau)
    return 1.0 / e.sum(axis=-1)


def run(binding, cfg, seqs=None, seed=synth.BASE_SEED, loss_floor=LOSS_FLOOR, grad_floor=GRAD_FLOOR):
    inp = synth.make_inputs(cfg, seed, sequences=seqs)
    T, D = dev(inp.target_logits), dev(inp.draft_logits)
    x, u = torch.from_numpy(inp.draft_tokens).cuda(), torch.from_numpy(inp.uniforms).cuda()
    out = binding.sd_verify_error_feedback(T, D, x, u, inp.tau)
    full = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    ref = sd_oracle.error_position_feedback(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms,
                                            inp.tau, nthreads=min(8, sd_oracle.max_threads()))
    tol = TOL[cfg.dtype]
    B, k, V = inp.target_logits.shape[0], cfg.k, cfg.V
    # the same verification as the full step, bit for bit
    assert torch.equal(out.accept_len, full.accept_len)
    assert torch.equal(out.tokens, full.tokens)
    assert torch.equal(out.loss, full.loss)
    assert torch.equal(out.status, full.status)
    n_gpu = out.accept_len.cpu().numpy()
    # against the oracle
    band = (ref.full.accept_band.sum(1) > 0) | (ref.full.cdf_margin <= 1e-6)
    assert (n_gpu[~band] == ref.full.accept_len[~band]).all()
    assert (out.tokens.cpu().numpy()[~band] == ref.full.tokens[~band]).all()
    loss = out.loss.cpu().numpy().astype(np.float64)
    assert (np.abs(loss - ref.full.loss) <= tol * np.maximum(np.abs(ref.full.loss), 1e-6) + loss_floor).all()
    g = out.error_grad.cpu().float().numpy().astype(np.float64)
    Tf, Df = f64(inp.target_logits), f64(inp.draft_logits)
    for b in range(B):
        n = int(n_gpu[b])
        if n == k:
            assert (g[b] == 0).all()
            continue
        want = ref.full.grad[b, n]
        bound = tol * np.abs(want).max() + grad_floor * max(pmax_of(Tf[b, n], inp.tau), pmax_of(Df[b, n], inp.tau)) / inp.tau
        assert np.abs(g[b] - want).max() <= bound, (b, n, np.abs(g[b] - want).max() / bound)
        # and the row is the full step's row of that position, bit for bit
        assert torch.equal(out.error_grad[b].view(torch.int16), full.grad_draft[b, n].view(torch.int16))
    return n_gpu


@pytest.mark.parametrize("name,seqs", [("cfg1", None), ("cfg2", None), ("cfg3", range(0, 32, 5)),
                                       ("cfg4", range(1, 64, 9)), ("cfg5", range(0, 256, 41))])
def test_workloads(binding, name, seqs):
    # the workloads at the contract's tolerance: no absolute term on the loss, no floor on the gradient
    run(binding, synth.CONFIGS[name], seqs=seqs, loss_floor=0.0, grad_floor=0.0)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,k,V", [(1, 1, 8), (3, 1, 1024), (5, 3, 70000), (41, 2, 2048), (2, 64, 520), (7, 5, 16392)])
def test_shapes(binding, dtype, B, k, V):
    run(binding, synth.custom_config(B, k, V, dtype=dtype, recipe="peaks", tau=0.8))


def test_every_accept_length_occurs_and_fully_accepted_rows_are_zero(binding):
    """Draft = target on a prefix of every sequence, far off behind it: accept lengths 0..k by design."""
    B, k, V = 12, 5, 4096
    cfg = synth.custom_config(B, k, V, dtype="f32")
    inp = synth.make_inputs(cfg)
    D = inp.draft_logits.copy()
    rng = np.random.default_rng(3)
    for b in range(B):
        n = b % (k + 1)
        D[b, :n] = inp.target_logits[b, :n]                 # ratio 1: always accepted
        if n < k:
            D[b, n] = -inp.target_logits[b, n]              # the draft's favourites are the target's least likely
            inp.draft_tokens[b, n] = int(np.argmax(D[b, n]))
            inp.uniforms[b, n] = 0.999
    inp.draft_logits[:] = D
    T, Dd = dev(inp.target_logits), dev(inp.draft_logits)
    x, u = torch.from_numpy(inp.draft_tokens).cuda(), torch.from_numpy(inp.uniforms).cuda()
    out = binding.sd_verify_error_feedback(T, Dd, x, u, inp.tau)
    torch.cuda.synchronize()
    ref = sd_oracle.error_position_feedback(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, inp.tau)
    n_gpu = out.accept_len.cpu().numpy()
    assert list(ref.full.accept_len) == [b % (k + 1) for b in range(B)]
    assert (n_gpu == ref.full.accept_len).all()
    g = out.error_grad.cpu().numpy().astype(np.float64)
    for b in range(B):
        if n_gpu[b] == k:
            assert (g[b] == 0).all()
        else:
            assert np.abs(g[b] - ref.error_grad[b]).max() <= 1e-5 * np.abs(ref.error_grad[b]).max() + 1e-6


@pytest.mark.parametrize("cluster", [1, 2, 3, 5, 8])
def test_every_cluster_size(binding, cluster, options):
    options(binding.SD_OPT_CLUSTER, cluster)
    run(binding, synth.custom_config(9, 3, 50000, dtype="bf16", tau=0.9))


def test_twice_in_a_row_and_between_other_entry_points(binding):
    cfg = synth.CONFIGS["cfg2"]
    a = run(binding, cfg)
    b = run(binding, cfg)
    assert (a == b).all()


def test_refusals(binding):
    cfg = synth.custom_config(2, 2, 1001, dtype="f32")          # rows are not whole 16-byte vectors
    inp = synth.make_inputs(cfg)
    with pytest.raises(binding.SdVerifyError):
        binding.sd_verify_error_feedback(dev(inp.target_logits), dev(inp.draft_logits),
                                         torch.from_numpy(inp.draft_tokens).cuda(),
                                         torch.from_numpy(inp.uniforms).cuda(), 1.0)


def test_full_size_bench_shape_equals_the_full_step(binding):
    """The bench shape (B=256, k=6, V=128256, fp32; 24-25 units per cluster, so every ring and every
    double-buffered slot of the kernel wraps many times): everything bit-equal to the full step, and
    a sample of sequences against the oracle."""
    cfg = synth.CONFIGS["cfg5"]
    inp = synth.make_inputs(cfg)
    T, D = dev(inp.target_logits), dev(inp.draft_logits)
    x, u = torch.from_numpy(inp.draft_tokens).cuda(), torch.from_numpy(inp.uniforms).cuda()
    out = binding.sd_verify_error_feedback(T, D, x, u, inp.tau)
    full = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    assert torch.equal(out.accept_len, full.accept_len)
    assert torch.equal(out.tokens, full.tokens)
    assert torch.equal(out.loss, full.loss)
    assert torch.equal(out.status, full.status)
    n = out.accept_len.long()
    rows = full.grad_draft[torch.arange(cfg.B, device="cuda"), n.clamp(max=cfg.k - 1)]
    rows[n == cfg.k] = 0
    assert torch.equal(out.error_grad, rows)
    seqs = np.array([0, 9, 77, 128, 201, 255])
    ref = sd_oracle.error_position_feedback(inp.target_logits[seqs], inp.draft_logits[seqs], inp.draft_tokens[seqs],
                                            inp.uniforms[seqs], inp.tau, nthreads=min(6, sd_oracle.max_threads()))
    safe = (ref.full.accept_band.sum(1) == 0) & (ref.full.cdf_margin > 1e-6)
    assert (out.accept_len.cpu().numpy()[seqs][safe] == ref.full.accept_len[safe]).all()
    assert (out.tokens.cpu().numpy()[seqs][safe] == ref.full.tokens[safe]).all()
    assert np.allclose(out.loss.cpu().numpy()[seqs], ref.full.loss, rtol=1e-5, atol=4e-7)
    g = out.error_grad.cpu().numpy()[seqs].astype(np.float64)
    for j in range(len(seqs)):
        if safe[j]:
            assert np.abs(g[j] - ref.error_grad[j]).max() <= 1e-5 * np.abs(ref.error_grad[j]).max() + 1e-7


@pytest.mark.parametrize("lag,cluster", [(0, 2), (2, 1), (100, 3), (1, 4)])
def test_orders_of_the_walk_and_cluster_sizes_with_many_units_per_cluster(binding, lag, cluster, options):
    """Many units per cluster (about 60 here) in every order of the walk: bit-equal to the full step
    run with the same settings."""
    options(binding.SD_OPT_LAG, lag)
    options(binding.SD_OPT_CLUSTER, cluster)
    cfg = synth.custom_config(600, 5, 8192, dtype="bf16", tau=0.9, recipe="peaks")
    inp = synth.make_inputs(cfg)
    T, D = dev(inp.target_logits), dev(inp.draft_logits)
    x, u = torch.from_numpy(inp.draft_tokens).cuda(), torch.from_numpy(inp.uniforms).cuda()
    out = binding.sd_verify_error_feedback(T, D, x, u, inp.tau)
    full = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    assert torch.equal(out.accept_len, full.accept_len)
    assert torch.equal(out.tokens, full.tokens)
    assert torch.equal(out.loss, full.loss)
    assert torch.equal(out.status, full.status)
    n = out.accept_len.long()
    rows = full.grad_draft[torch.arange(cfg.B, device="cuda"), n.clamp(max=cfg.k - 1)]
    rows[n == cfg.k] = 0
    assert torch.equal(out.error_grad.view(torch.int16), rows.view(torch.int16))


def test_optional_outputs_can_be_left_out(binding):
    cfg = synth.CONFIGS["cfg2"]
    inp = synth.make_inputs(cfg)
    T, D = dev(inp.target_logits), dev(inp.draft_logits)
    x, u = torch.from_numpy(inp.draft_tokens).cuda(), torch.from_numpy(inp.uniforms).cuda()
    full = binding.sd_verify_error_feedback(T, D, x, u, inp.tau)
    for kw in (dict(want_loss=False), dict(want_grad=False), dict(want_status=False),
               dict(want_loss=False, want_grad=False, want_status=False)):
        out = binding.sd_verify_error_feedback(T, D, x, u, inp.tau, **kw)
        torch.cuda.synchronize()
        assert torch.equal(out.accept_len, full.accept_len) and torch.equal(out.tokens, full.tokens)
        if out.loss is not None:
            assert torch.equal(out.loss, full.loss)
        if out.error_grad is not None:
            assert torch.equal(out.error_grad.view(torch.int16), full.error_grad.view(torch.int16))
