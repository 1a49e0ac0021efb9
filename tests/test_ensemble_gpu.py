"""GPU parity of the online-ensemble feedback (Sec. 3.3) against the CPU oracle: per-learner loss
and gradient within the tolerances of the single-draft step, the round's mean loss, the cumulative
losses and the Hedge weights.

Bars: loss |gpu - ref| <= tol*|ref| + 4e-7 with tol = 1e-5 (fp32 logits) / 2e-2 (bf16 logits);
gradient per row max|gpu - ref| <= tol*max|ref| + 8*2^-24*max(p,q)/tau; mean loss of the round and
cumulative loss like the loss; a weight is exp(-eps*cum)/Z, so its relative error is at most
2*eps times the absolute error of the cumulative losses, plus fp32 rounding of the stored weight.
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
EPS = 10.0


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


def compare(inp, Ds, out, ref, cum_in=None, eps=EPS, loss_floor=LOSS_FLOOR, grad_floor=GRAD_FLOOR):
    tol = TOL[inp.cfg.dtype]
    k = inp.cfg.k
    loss = out.loss.cpu().numpy().astype(np.float64)
    err = np.abs(loss - ref.loss)
    bound = tol * np.maximum(np.abs(ref.loss), 1e-6) + loss_floor
    assert (err <= bound).all(), f"loss: worst ratio {np.max(err / bound):.3g}"
    if out.grad is not None:
        pm = pmax_of(f64(inp.target_logits)[:, :k], inp.tau)
        for n, D in enumerate(Ds):
            g = out.grad[n].cpu().float().numpy().astype(np.float64)
            qm = pmax_of(f64(D), inp.tau)
            worst = np.abs(g - ref.grad[n]).max(axis=2)
            gb = tol * np.abs(ref.grad[n]).max(axis=2) + grad_floor * np.maximum(pm, qm) / inp.tau
            assert (worst <= gb).all(), f"grad of learner {n}: worst ratio {np.max(worst / gb):.3g}"
    rl = out.round_loss.cpu().numpy()
    cum = out.cum_loss.cpu().numpy()
    w = out.weights.cpu().numpy().astype(np.float64)
    lb = tol * np.maximum(np.abs(ref.round_loss), 1e-6) + loss_floor
    assert (np.abs(rl - ref.round_loss) <= lb).all()
    assert (np.abs(cum - ref.cum_loss) <= lb + 1e-15 * np.abs(ref.cum_loss)).all()
    assert abs(w.sum() - 1.0) < 1e-6
    assert (np.abs(w - ref.weights) <= 2 * eps * lb.max() * ref.weights + 2.0 ** -23).all(), (w, ref.weights)
    # the device's own weights are the exponential weighting of the device's own cumulative losses
    mine = np.exp(-eps * (cum - cum.min()))
    np.testing.assert_allclose(w, mine / mine.sum(), rtol=3e-7, atol=1e-12)


def run(binding, cfg, N=3, seqs=None, cum_in=None, want_grad=True, eps=EPS, **floors):
    inp = synth.make_inputs(cfg, sequences=seqs)
    Ds = synth.ensemble_drafts(inp, N)
    ref = sd_oracle.ensemble_feedback(inp.target_logits, Ds, inp.tau, eps, cum_loss=cum_in, want_grad=want_grad,
                                      nthreads=min(8, sd_oracle.max_threads()))
    cum_dev = None if cum_in is None else torch.from_numpy(np.asarray(cum_in, np.float64)).cuda()
    out = binding.sd_ensemble_feedback(dev(inp.target_logits), [dev(d) for d in Ds], inp.tau, eps,
                                       cum_loss=cum_dev, want_grad=want_grad, want_status=True)
    torch.cuda.synchronize()
    assert (out.status.cpu().numpy() == 0).all()
    compare(inp, Ds, out, ref, cum_in, eps, **floors)
    return inp, Ds, out, ref


@pytest.mark.parametrize("name,seqs", [("cfg1", None), ("cfg2", None), ("cfg3", range(0, 32, 11)),
                                       ("cfg4", range(2, 64, 23)), ("cfg5", range(0, 256, 97))])
def test_workloads_three_learners(binding, name, seqs):
    # the workloads at the contract's tolerance: no absolute term on the loss, no floor on the gradient
    run(binding, synth.CONFIGS[name], N=3, seqs=seqs, cum_in=[0.3, 0.1, 0.2], loss_floor=0.0, grad_floor=0.0)


@pytest.mark.parametrize("N", [1, 2, 5, 8])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_number_of_learners(binding, N, dtype):
    cfg = synth.custom_config(5, 3, 4096 + 8 * 37, dtype=dtype, tau=0.8, recipe="peaks")
    run(binding, cfg, N=N)


@pytest.mark.parametrize("B,k,V", [(1, 1, 8), (2, 1, 1024), (3, 4, 70000), (37, 2, 2048), (2, 64, 520)])
def test_shapes(binding, B, k, V):
    run(binding, synth.custom_config(B, k, V, dtype="f32"), N=3)
    run(binding, synth.custom_config(B, k, V, dtype="bf16"), N=2, want_grad=False)


@pytest.mark.parametrize("cluster", [1, 2, 3, 4, 6, 8])
def test_every_cluster_size(binding, cluster, options):
    options(binding.SD_OPT_CLUSTER, cluster)
    cfg = synth.custom_config(6, 3, 50000, dtype="f32", tau=0.9)
    run(binding, cfg, N=3)
    assert binding.sd_launch_info()["cluster_size"] == cluster


def test_each_learner_equals_the_single_draft_step_bit_for_bit(binding, options):
    """The units of the ensemble run the arithmetic of the single-draft step: at the same cluster
    size the same loss bits and the same gradient bits, whichever learner and wherever the unit
    falls in a cluster's range."""
    options(binding.SD_OPT_CLUSTER, 2)
    cfg = synth.CONFIGS["cfg2"]
    inp = synth.make_inputs(cfg)
    Ds = synth.ensemble_drafts(inp, 3)
    T = dev(inp.target_logits)
    x = torch.from_numpy(inp.draft_tokens).cuda()
    u = torch.from_numpy(inp.uniforms).cuda()
    out = binding.sd_ensemble_feedback(T, [dev(d) for d in Ds], inp.tau, EPS)
    for n, D in enumerate(Ds):
        one = binding.sd_verify_feedback(T, dev(D), x, u, inp.tau)
        torch.cuda.synchronize()
        assert torch.equal(one.loss, out.loss[n])
        assert torch.equal(one.grad_draft.view(torch.int16), out.grad[n].view(torch.int16))


def test_rounds_accumulate_in_place_and_weights_track_the_best_learner(binding):
    cfg = synth.custom_config(4, 3, 8192, dtype="bf16", tau=1.0)
    cum = torch.zeros(3, dtype=torch.float64, device="cuda")
    total = np.zeros(3)
    out = None
    for rnd in range(4):
        inp = synth.make_inputs(cfg, seed=synth.BASE_SEED + rnd)
        Ds = synth.ensemble_drafts(inp, 3, seed=synth.BASE_SEED + rnd)
        ref = sd_oracle.ensemble_feedback(inp.target_logits, Ds, inp.tau, EPS, cum_loss=total, want_grad=False)
        out = binding.sd_ensemble_feedback(dev(inp.target_logits), [dev(d) for d in Ds], inp.tau, EPS,
                                           cum_loss=cum, want_grad=False)
        torch.cuda.synchronize()
        total = ref.cum_loss
        cum = out.cum_loss                        # feeds the next round
        np.testing.assert_allclose(out.cum_loss.cpu().numpy(), total, rtol=1e-5)
    w = out.weights.cpu().numpy()
    assert w[0] > 0.99 or w.argmax() == int(np.argmin(total))


def test_refusals(binding):
    cfg = synth.custom_config(2, 2, 1001, dtype="f32")          # rows are not whole 16-byte vectors
    inp = synth.make_inputs(cfg)
    with pytest.raises(binding.SdVerifyError):
        binding.sd_ensemble_feedback(dev(inp.target_logits), [dev(inp.draft_logits)], 1.0, EPS)
    cfg = synth.custom_config(2, 2, 1024, dtype="f32")
    inp = synth.make_inputs(cfg)
    T, D = dev(inp.target_logits), dev(inp.draft_logits)
    with pytest.raises(binding.SdVerifyError):
        binding.sd_ensemble_feedback(T, [D] * 9, 1.0, EPS)        # more learners than SD_MAX_LEARNERS
    with pytest.raises(binding.SdVerifyError):
        binding.sd_ensemble_feedback(T, [D], 0.0, EPS)
    with pytest.raises(binding.SdVerifyError):
        binding.sd_ensemble_feedback(T, [D], 1.0, -1.0)
    # and the library still works afterwards
    out = binding.sd_ensemble_feedback(T, [D, T[:, :2].contiguous()], 1.0, EPS)
    torch.cuda.synchronize()
    assert float(out.round_loss[1]) < 1e-9 and float(out.weights[1]) > float(out.weights[0])


def test_full_size_bench_shape_equals_the_single_draft_step(binding, options):
    """The bench shape with 3 learners (B=256, k=6, V=128256, fp32; 62 units per cluster): every
    learner's loss and gradient bit-equal to the single-draft step on the same logits, and the
    weights from the device's own losses."""
    options(binding.SD_OPT_CLUSTER, 2)
    cfg = synth.CONFIGS["cfg5"]
    inp = synth.make_inputs(cfg)
    Ds = synth.ensemble_drafts(inp, 3)
    T = dev(inp.target_logits)
    x = torch.from_numpy(inp.draft_tokens).cuda()
    u = torch.from_numpy(inp.uniforms).cuda()
    dDs = [dev(d) for d in Ds]
    out = binding.sd_ensemble_feedback(T, dDs, inp.tau, EPS, want_status=True)
    torch.cuda.synchronize()
    assert (out.status.cpu().numpy() == 0).all()
    for n in range(3):
        one = binding.sd_verify_feedback(T, dDs[n], x, u, inp.tau)
        torch.cuda.synchronize()
        assert torch.equal(one.loss, out.loss[n])
        assert torch.equal(one.grad_draft, out.grad[n])
        del one
    mean = out.loss.double().mean(dim=(1, 2)).cpu().numpy()
    np.testing.assert_allclose(out.round_loss.cpu().numpy(), mean, rtol=1e-12)
    w = np.exp(-EPS * (mean - mean.min()))
    np.testing.assert_allclose(out.weights.cpu().numpy(), w / w.sum(), rtol=3e-7, atol=1e-12)


@pytest.mark.parametrize("lag,cluster", [(0, 2), (2, 1), (100, 3)])
def test_orders_of_the_walk_with_many_units_per_cluster(binding, lag, cluster, options):
    options(binding.SD_OPT_LAG, lag)
    options(binding.SD_OPT_CLUSTER, cluster)
    cfg = synth.custom_config(300, 4, 8192, dtype="bf16", tau=0.9, recipe="peaks")
    inp = synth.make_inputs(cfg)
    Ds = synth.ensemble_drafts(inp, 3)
    T = dev(inp.target_logits)
    x = torch.from_numpy(inp.draft_tokens).cuda()
    u = torch.from_numpy(inp.uniforms).cuda()
    dDs = [dev(d) for d in Ds]
    out = binding.sd_ensemble_feedback(T, dDs, inp.tau, EPS)
    for n in range(3):
        one = binding.sd_verify_feedback(T, dDs[n], x, u, inp.tau)
        torch.cuda.synchronize()
        assert torch.equal(one.loss, out.loss[n])
        assert torch.equal(one.grad_draft.view(torch.int16), out.grad[n].view(torch.int16))


def test_gradients_of_some_learners_can_be_left_out(binding):
    """A NULL entry in the array of gradient pointers: no gradient for that learner, the rest unchanged."""
    import ctypes
    cfg = synth.custom_config(4, 3, 8192, dtype="f32")
    inp = synth.make_inputs(cfg)
    Ds = synth.ensemble_drafts(inp, 3)
    T, dDs = dev(inp.target_logits), [dev(d) for d in Ds]
    full = binding.sd_ensemble_feedback(T, dDs, inp.tau, EPS)
    torch.cuda.synchronize()
    out = binding.EnsembleOutputs(loss=torch.empty_like(full.loss), grad=None,
                                  round_loss=torch.empty_like(full.round_loss), cum_loss=torch.empty_like(full.cum_loss),
                                  weights=torch.empty_like(full.weights), status=None)
    g0 = torch.full_like(full.grad[0], 7.0)
    g2 = torch.empty_like(full.grad[2])
    dptr = (ctypes.c_void_p * 3)(*[d.data_ptr() for d in dDs])
    gptr = (ctypes.c_void_p * 3)(None, None, g2.data_ptr())
    rc = binding._lib.sd_ensemble_feedback(T.data_ptr(), dptr, 3, float(inp.tau), EPS, cfg.B, cfg.k, cfg.V, 0, None,
                                           out.loss.data_ptr(), gptr, out.round_loss.data_ptr(),
                                           out.cum_loss.data_ptr(), out.weights.data_ptr(), None, None, 0, None)
    torch.cuda.synchronize()
    assert rc == 0
    assert torch.equal(out.loss, full.loss) and torch.equal(out.weights, full.weights)
    assert torch.equal(g2, full.grad[2]) and (g0 == 7.0).all()
