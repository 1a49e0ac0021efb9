"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs and the same pre-drawn uniforms.

Bars (stated here, derived in the design notes):
  * accept lengths and emitted tokens are bit-exact, except for sequences the oracle marks as
    sitting on a decision threshold: a reached accept test with |u - p/q| < 1e-6, or an
    inverse-CDF draw whose target lies within 1e-6 (relative to the total mass) of an interval
    edge.  Those sequences are counted, must be rare, and must still produce a valid answer.
  * loss: on the five workloads |gpu - ref| <= tol * max(|ref|, 1e-6), tol = 1e-5 (fp32 logits) /
    2e-2 (bf16 logits), nothing added.  The edge-case tests (rows with KL near zero: identical or
    nearly identical models, tiny vocabularies) add an absolute 4e-7, the rounding floor of the
    method in fp32: KL is log S_D - log S_T plus a mean, and each softmax denominator S carries a
    relative error of a few 2^-24 (2^-22 per term from the hardware exp2, averaged over the row),
    whatever the size of KL.
  * gradient, per row: max|gpu - ref| <= tol * max|ref| + floor and the same in the L2 norm, the
    reference being the fp64 value before any rounding to bf16.  floor = 8 * 2^-24 * max(p,q)/tau
    is the rounding of p and q themselves: it only matters when q - p is a difference of two
    nearly equal large probabilities (near one-hot rows); the five workloads are checked without it.
  * inside the band a sequence may differ from the oracle's answer only in the way the band
    allows: the accept lengths part at a flagged test, and the extra token is one whose interval
    of the oracle's inverse CDF (for the accept length the device took) lies within 1e-6 of the
    total mass from u_k times the total mass.
"""
import os

import numpy as np
import pytest
import torch

from oracle import sd_oracle
from paper_2603_12617_b200 import synth

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-2}
LOSS_FLOOR = 4e-7
GRAD_FLOOR = 8 * 2.0 ** -24


def logits_f64(inp, seqs=None):
    sl = slice(None) if seqs is None else np.asarray(seqs)
    T, D = inp.target_logits[sl], inp.draft_logits[sl]
    if inp.cfg.dtype == "bf16":
        T, D = synth.bf16_bits_to_f32(T), synth.bf16_bits_to_f32(D)
    return T.astype(np.float64), D.astype(np.float64)


def prob_max_and_l2(z, tau):
    """Largest softmax probability and L2 norm of the softmax of every row of z[..., V]."""
    e = np.exp((z - z.max(axis=-1, keepdims=True)) / tau)
    s = e.sum(axis=-1)
    return 1.0 / s, np.sqrt((e * e).sum(axis=-1)) / s


@pytest.fixture(scope="module")
def binding():
    import __graft_entry__ as entry
    entry.build()
    from paper_2603_12617_b200 import binding as b
    return b


def to_device(inp):
    T = torch.from_numpy(inp.target_logits).cuda()
    D = torch.from_numpy(inp.draft_logits).cuda()
    if inp.cfg.dtype == "bf16":
        T, D = T.view(torch.bfloat16), D.view(torch.bfloat16)
    return T, D, torch.from_numpy(inp.draft_tokens).cuda(), torch.from_numpy(inp.uniforms).cuda()


def oracle_of(inp, seqs=None, want_grad=True):
    sl = slice(None) if seqs is None else np.asarray(seqs)
    return sd_oracle.verify_feedback(inp.target_logits[sl], inp.draft_logits[sl], inp.draft_tokens[sl],
                                     inp.uniforms[sl], inp.tau, want_grad=want_grad,
                                     nthreads=min(8, sd_oracle.max_threads()))


BAND = 1e-6
COUNTS = {}     # per workload: what the five-workload tests print at the end


def check_band_answer(inp, b_global, n_gpu, tok_gpu, ref, j):
    """A sequence whose answer differs from the oracle's: it must be one the threshold band allows."""
    k = inp.cfg.k
    n_ref = int(ref.accept_len[j])
    if n_gpu != n_ref:
        first = min(n_gpu, n_ref)
        assert first < k and ref.accept_band[j, first], \
            f"sequence {b_global}: accept length {n_gpu} vs {n_ref} without a flagged test at position {first}"
    y = int(tok_gpu[n_gpu])
    lo, hi, R = sd_oracle.draw_interval(inp.target_logits[b_global], inp.draft_logits[b_global], inp.tau, n_gpu, y)
    t = float(inp.uniforms[b_global, k]) * R
    assert hi > lo, f"sequence {b_global}: token {y} has no mass in the distribution it was drawn from"
    assert lo - BAND * R <= t <= hi + BAND * R, \
        f"sequence {b_global}: token {y} owns [{lo / R:.9f}, {hi / R:.9f}) of the CDF, u_k = {t / R:.9f}"


def check(inp, out, ref, seqs=None, max_band_frac=0.02, check_grad=True, check_loss=True,
          loss_floor=LOSS_FLOOR, grad_floor=GRAD_FLOOR):
    """Compare device outputs (for sequences `seqs`, default all) with the oracle's."""
    dtype = inp.cfg.dtype
    tol = TOL[dtype]
    idx = np.arange(ref.tokens.shape[0]) if seqs is None else np.asarray(seqs)
    sl = torch.as_tensor(idx)
    n_gpu = out.accept_len.cpu()[sl].numpy()
    tok_gpu = out.tokens.cpu()[sl].numpy()
    B, k, V = ref.tokens.shape[0], inp.cfg.k, inp.cfg.V
    x = inp.draft_tokens[idx]

    # A draw that lands in a token of mass < 2e-6 is inside the sample band by construction, so with
    # V > 10^5 the band itself is not rare; what must be rare is a disagreement, and every
    # disagreement must sit inside the band and be an answer the band allows.
    accept_band = ref.accept_band.sum(1) > 0
    sample_band = ref.cdf_margin <= BAND
    band = accept_band | sample_band
    safe = ~band
    assert (n_gpu[safe] == ref.accept_len[safe]).all(), "accept lengths differ off the threshold band"
    assert (tok_gpu[safe] == ref.tokens[safe]).all(), "emitted tokens differ off the threshold band"
    mismatch = (n_gpu != ref.accept_len) | (tok_gpu != ref.tokens).any(axis=1)
    assert mismatch.sum() <= max(1, int(max_band_frac * B)), \
        f"{mismatch.sum()} of {B} sequences differ inside the threshold band ({band.sum()} in the band)"
    assert ref.accept_band.sum() <= max(1, int(max_band_frac * B * k)), "accept band is not rare"
    # every sequence, band or not, has a well-formed answer
    assert ((n_gpu >= 0) & (n_gpu <= k)).all()
    for j in range(B):
        n = int(n_gpu[j])
        assert (tok_gpu[j, :n] == x[j, :n]).all()
        assert 0 <= tok_gpu[j, n] < V
        assert (tok_gpu[j, n + 1:] == -1).all()
    for j in np.nonzero(mismatch)[0]:
        check_band_answer(inp, int(idx[j]), int(n_gpu[j]), tok_gpu[j], ref, int(j))

    if check_loss and out.loss is not None:
        loss = out.loss.cpu()[sl].numpy().astype(np.float64)
        err = np.abs(loss - ref.loss)
        bound = tol * np.maximum(np.abs(ref.loss), 1e-6) + loss_floor
        ok = (err <= bound) | (loss == ref.loss)          # the second term covers +inf == +inf
        assert ok.all(), f"loss: worst ratio {np.nanmax(err / bound):.3g}"
    if check_grad and out.grad_draft is not None and ref.grad is not None:
        g = out.grad_draft.cpu()[sl].float().numpy().astype(np.float64)
        d = g - ref.grad
        T64, D64 = logits_f64(inp, idx)
        pmax, p2 = prob_max_and_l2(T64[:, :k], inp.tau)
        qmax, q2 = prob_max_and_l2(D64, inp.tau)
        gmax = np.abs(ref.grad).max(axis=2)
        bound = tol * gmax + grad_floor * np.maximum(pmax, qmax) / inp.tau
        worst = np.abs(d).max(axis=2)
        assert (worst <= bound).all(), f"grad max-norm: worst ratio {np.max(worst / bound):.3g}"
        l2 = np.sqrt((d * d).sum(axis=2))
        ref_l2 = np.sqrt((ref.grad * ref.grad).sum(axis=2))
        assert (l2 <= tol * ref_l2 + grad_floor * (p2 + q2) / inp.tau).all(), "grad L2 norm"
    if out.acc_prob is not None:
        acc = out.acc_prob.cpu()[sl].numpy().astype(np.float64)
        assert np.abs(acc - ref.acc_prob).max() < 2e-5
    if out.status is not None:
        assert (out.status.cpu()[sl].numpy() == ref.status.astype(np.int32)).all()
    return {"sequences": int(B), "accept_band_rows": int(ref.accept_band.sum()),
            "sample_band_rows": int(sample_band.sum()), "mismatches": int(mismatch.sum()),
            "mean_accept_len": float(n_gpu.mean()), "mean_acc_prob": float(ref.acc_prob.mean())}


def add_counts(name, c):
    t = COUNTS.setdefault(name, {"sequences": 0, "accept_band_rows": 0, "sample_band_rows": 0, "mismatches": 0,
                                 "accept_len_sum": 0.0, "acc_prob_sum": 0.0})
    for key in ("sequences", "accept_band_rows", "sample_band_rows", "mismatches"):
        t[key] += c[key]
    t["accept_len_sum"] += c["mean_accept_len"] * c["sequences"]
    t["acc_prob_sum"] += c["mean_acc_prob"] * c["sequences"]
    print(f"[parity] {name}: {t['sequences']} sequences compared, accept-band rows {t['accept_band_rows']}, "
          f"sample-band rows {t['sample_band_rows']}, mismatches (all inside the band, all valid) {t['mismatches']}, "
          f"mean accept length {t['accept_len_sum'] / t['sequences']:.3f}, "
          f"mean sum min(p,q) {t['acc_prob_sum'] / t['sequences']:.4f}")


def run_and_check(binding, cfg, seed=synth.BASE_SEED, ex=False, **kw):
    inp = synth.make_inputs(cfg, seed)
    T, D, x, u = to_device(inp)
    out = (binding.sd_verify_feedback_ex if ex else binding.sd_verify_feedback)(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    ref = oracle_of(inp)
    counts = check(inp, out, ref, **kw)
    return inp, out, ref, counts


# ------------------------------------------------------------------ the five workloads
@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4"])
@pytest.mark.parametrize("seed_off", [0, 1])
def test_config_full_parity(binding, name, seed_off):
    """Every sequence of the workload, both seeds, at the tolerance the contract states: no
    absolute term on the loss, no floor on the gradient."""
    cfg = synth.CONFIGS[name]
    inp, out, ref, counts = run_and_check(binding, cfg, synth.BASE_SEED + seed_off, ex=True,
                                          loss_floor=0.0, grad_floor=0.0)
    add_counts(f"{name} seed+{seed_off}", counts)
    info = binding.sd_launch_info()
    assert info["path"] == 1, "the five workloads must take the cluster fast path"


def test_config5_full_size_every_sequence(binding):
    """B=256, k=6, V=128256 fp32 in the launch configuration the benchmark times, every sequence
    against the oracle element by element (in slices of 32 sequences: the fp64 gradient of a slice
    is 0.2 GB), at the contract's tolerance without floors."""
    cfg = synth.CONFIGS["cfg5"]
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)
    out = binding.sd_verify_feedback(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    assert binding.sd_launch_info()["path"] == 1
    acc_sum = 0.0
    for b0 in range(0, cfg.B, 32):
        seqs = list(range(b0, min(cfg.B, b0 + 32)))
        ref = oracle_of(inp, seqs)
        counts = check(inp, out, ref, seqs=seqs, max_band_frac=0.1, loss_floor=0.0, grad_floor=0.0)
        add_counts("cfg5", counts)
        acc_sum += ref.acc_prob.sum()
        del ref
    n = out.accept_len.cpu().numpy()
    gsum = out.grad_draft.sum(dim=2).abs().max().item()
    assert gsum < 1e-4                     # rows of (q-p)/tau sum to zero
    # expected mean accepted length from the closed form of the proof of Lemma 1, with the
    # per-position acceptance probabilities of the workload
    acc = acc_sum / (cfg.B * cfg.k)
    expect = (1 - acc ** (cfg.k + 1)) / (1 - acc)
    assert abs((n + 1).mean() - expect) < 0.35


# ------------------------------------------------------------------ shapes and alignments
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,k,V", [(1, 1, 5), (2, 3, 17), (3, 2, 1023), (2, 2, 4100), (1, 1, 8), (2, 2, 512),
                                   (3, 1, 520), (2, 4, 1024), (1, 2, 40000), (5, 3, 2056)])
def test_shapes(binding, dtype, B, k, V):
    cfg = synth.custom_config(B=B, k=k, V=V, dtype=dtype, tau=0.85, index=50)
    run_and_check(binding, cfg, ex=True, max_band_frac=1.0)


def test_largest_k(binding):
    cfg = synth.custom_config(B=2, k=64, V=1000, dtype="f32", d_sigma=0.1, index=51)
    run_and_check(binding, cfg, ex=True, max_band_frac=1.0)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("cluster", [1, 2, 3, 4, 5, 6, 7, 8])
def test_every_cluster_size_gives_the_same_answer(binding, dtype, cluster, options):
    cfg = synth.custom_config(B=3, k=3, V=24000 if dtype == "f32" else 48000, dtype=dtype, tau=1.2, index=52)
    options(binding.SD_OPT_CLUSTER, cluster)
    inp, out, ref, _ = run_and_check(binding, cfg, ex=True, max_band_frac=1.0)
    info = binding.sd_launch_info()
    assert info["path"] == 1 and info["cluster_size"] == cluster


@pytest.mark.parametrize("lag", [0, 1, 2, 100, -2])
@pytest.mark.parametrize("cluster", [1, 3, 4, 8])
def test_every_order_of_the_two_passes_gives_the_same_answer(binding, lag, cluster, options):
    """Pass 2 of a unit may come 0, 1, 2 ... stages (per warp) into pass 1 of the next unit, or after
    all of it (or both, cluster by cluster); several units per cluster, slices of 1 to 7 stages."""
    cfg = synth.custom_config(B=40, k=3, V=100000, dtype="bf16", tau=1.1, index=65)
    options(binding.SD_OPT_CLUSTER, cluster)
    options(binding.SD_OPT_LAG, lag)
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    info = binding.sd_launch_info()
    assert info["path"] == 1 and info["cluster_size"] == cluster
    seqs = [0, 1, 13, 26, 39]
    check(inp, out, oracle_of(inp, seqs), seqs=seqs, max_band_frac=1.0)
    base = getattr(test_every_order_of_the_two_passes_gives_the_same_answer, "_base", None)
    key = (cluster,)
    if base is None or key not in base:
        base = base or {}
        base[key] = out
        test_every_order_of_the_two_passes_gives_the_same_answer._base = base
    else:   # the order of the passes changes no bit of any output
        ref = base[key]
        assert torch.equal(ref.accept_len, out.accept_len) and torch.equal(ref.tokens, out.tokens)
        assert torch.equal(ref.loss, out.loss)
        assert torch.equal(ref.grad_draft.view(torch.int16), out.grad_draft.view(torch.int16))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_generic_path_matches_fast_path(binding, dtype, options):
    cfg = synth.custom_config(B=3, k=3, V=20000, dtype=dtype, tau=0.9, index=53)
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)
    fast = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    assert binding.sd_launch_info()["path"] == 1
    options(binding.SD_OPT_FORCE_GENERIC, 1)
    slow = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    assert binding.sd_launch_info()["path"] == 0
    ref = oracle_of(inp)
    check(inp, slow, ref, max_band_frac=1.0)
    assert (fast.accept_len == slow.accept_len).all() and (fast.tokens == slow.tokens).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_misaligned_base_pointers(binding, dtype):
    """Tensors that start one element past a 16-byte boundary take the generic path."""
    cfg = synth.custom_config(B=2, k=2, V=4096, dtype=dtype, index=54)
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)

    def shifted(t):
        buf = torch.empty(t.numel() + 1, dtype=t.dtype, device=t.device)
        v = buf[1:].view(t.shape)
        v.copy_(t)
        return v

    Ts, Ds = shifted(T), shifted(D)
    out = binding.sd_verify_feedback_ex(Ts, Ds, x, u, inp.tau)
    torch.cuda.synchronize()
    assert binding.sd_launch_info()["path"] == 0
    check(inp, out, oracle_of(inp), max_band_frac=1.0)


# ------------------------------------------------------------------ values
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_identical_models(binding, dtype):
    """p = q: everything accepted, zero loss, zero gradient (check 3 of the contract)."""
    cfg = synth.custom_config(B=4, k=5, V=32000, dtype=dtype, tau=0.7, index=55)
    inp = synth.make_inputs(cfg)
    inp.draft_logits[:] = inp.target_logits[:, :cfg.k]
    T, D, x, u = to_device(inp)
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    assert (out.accept_len.cpu() == cfg.k).all()
    assert out.loss.abs().max().item() == 0.0
    # q - p is evaluated as fma(eD, kD, -(eT*kT)): with identical rows that leaves the rounding
    # residual of one product, far below one ulp of p
    T64, _ = logits_f64(inp)
    pmax, _ = prob_max_and_l2(T64[:, :cfg.k], inp.tau)
    gabs = out.grad_draft.float().abs().amax(dim=2).cpu().numpy()
    assert (gabs <= 2.0 ** -24 * pmax / inp.tau).all()
    assert (out.acc_prob.cpu() - 1).abs().max().item() < 1e-6
    check(inp, out, oracle_of(inp), max_band_frac=1.0)


def test_shifted_and_huge_logits(binding):
    """Max-subtraction: +80 / -80 offsets and a spread that overflows a naive exp."""
    cfg = synth.custom_config(B=3, k=2, V=3000, dtype="f32", t_sigma=20.0, d_sigma=2.0, index=56)
    inp = synth.make_inputs(cfg)
    inp.target_logits[0] += 80.0
    inp.draft_logits[0] -= 80.0
    inp.target_logits[1] *= 4.0
    T, D, x, u = to_device(inp)
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    check(inp, out, oracle_of(inp), max_band_frac=1.0)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_late_spike_far_above_everything_seen(binding, dtype, options):
    """A logit that towers over all earlier ones late in a row: the fast path works with the
    references it has and must notice that this stage needs new ones."""
    options(binding.SD_OPT_CLUSTER, 1)          # one block per row: many stages per warp
    cfg = synth.custom_config(B=3, k=2, V=131072, dtype=dtype, t_sigma=1.0, d_sigma=0.5, index=64)
    inp = synth.make_inputs(cfg)
    big = np.float32(300.0) if dtype == "f32" else synth.f32_to_bf16_bits(np.array([300.0], np.float32))[0]
    inp.target_logits[0, 0, 120000] = big                  # target only
    inp.draft_logits[1, 1, 99999] = big                    # draft only
    inp.target_logits[2, 1, 70001] = big                   # both, different places
    inp.draft_logits[2, 1, 130000] = big
    inp.target_logits[2, 2, 131071] = big                  # bonus row, last entry
    T, D, x, u = to_device(inp)
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    assert binding.sd_launch_info()["path"] == 1
    check(inp, out, oracle_of(inp), max_band_frac=1.0)


def test_all_equal_logits(binding):
    cfg = synth.custom_config(B=2, k=2, V=777, dtype="f32", index=57)
    inp = synth.make_inputs(cfg)
    inp.target_logits[:] = 1.5
    inp.draft_logits[:] = -0.25
    T, D, x, u = to_device(inp)
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    ref = oracle_of(inp)
    assert (out.accept_len.cpu().numpy() == cfg.k).all()
    assert out.loss.abs().max().item() < 1e-6
    # uniform distribution: token index = floor(u*V) up to the edge band
    check(inp, out, ref, max_band_frac=1.0)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_masked_vocabulary_entries(binding, dtype):
    """-inf logits (masked tokens) in either model."""
    cfg = synth.custom_config(B=3, k=3, V=8192, dtype=dtype, index=58)
    inp = synth.make_inputs(cfg)
    ninf = np.float32(-np.inf) if dtype == "f32" else np.uint16(0xFF80)
    inp.target_logits[:, :, 100:4000] = ninf          # whole vectors and chunks masked
    inp.draft_logits[:, :, 100:3000] = ninf
    inp.draft_tokens[:] = np.clip(inp.draft_tokens, 4000, None)
    inp.draft_tokens[0, 0] = 3500                      # p(x) = 0, q(x) > 0: rejected
    T, D, x, u = to_device(inp)
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    ref = oracle_of(inp)
    assert out.accept_len.cpu()[0].item() == 0
    assert np.isfinite(ref.loss).all()
    check(inp, out, ref, max_band_frac=1.0)


def test_infinite_divergence(binding):
    cfg = synth.custom_config(B=1, k=1, V=1024, dtype="f32", index=59)
    inp = synth.make_inputs(cfg)
    inp.draft_logits[0, 0, 5] = -np.inf               # q = 0 where p > 0
    inp.draft_tokens[0, 0] = 7
    T, D, x, u = to_device(inp)
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    assert torch.isinf(out.loss[0, 0]).item() and out.loss[0, 0].item() > 0
    assert np.isinf(oracle_of(inp).loss[0, 0])


def test_bad_token_sets_status(binding):
    cfg = synth.custom_config(B=3, k=3, V=2048, dtype="f32", d_sigma=0.01, index=60)
    inp = synth.make_inputs(cfg)
    inp.draft_tokens[1, 1] = cfg.V
    inp.draft_tokens[2, 0] = -3
    T, D, x, u = to_device(inp)
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    st = out.status.cpu().numpy()
    ref = oracle_of(inp)
    assert st[0] == 0 and st[1] & binding.SD_STATUS_BAD_TOKEN and st[2] & binding.SD_STATUS_BAD_TOKEN
    assert out.accept_len.cpu().numpy()[2] == 0 and out.accept_len.cpu().numpy()[1] <= 1
    check(inp, out, ref, max_band_frac=1.0)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [4096, 777])
def test_zero_residual_at_a_forced_rejection(binding, dtype, V):
    """q = p exactly and a draft token outside the vocabulary: the rejection leaves a residual
    without mass, and the extra token is drawn from p_n instead (status BAD_TOKEN | ZERO_RESIDUAL).
    With all logits zero every product in the gradient is exact, so the device sees a residual of
    exactly zero as well and takes its own fallback (a draw over the whole row by one warp);
    V = 4096 goes through the cluster path, V = 777 through the element-wise one."""
    cfg = synth.custom_config(B=6, k=3, V=V, dtype=dtype, tau=0.9, index=66)
    inp = synth.make_inputs(cfg)
    inp.target_logits[:] = 0
    inp.draft_logits[:] = 0
    inp.draft_tokens[1, 1] = V            # rejected at position 1
    inp.draft_tokens[2, 0] = -1           # rejected at position 0
    inp.draft_tokens[4, 2] = V + 5        # rejected at the last position
    T, D, x, u = to_device(inp)
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    ref = oracle_of(inp)
    assert ref.status.tolist() == [0, 5, 5, 0, 5, 0]
    assert ref.accept_len.tolist() == [3, 1, 0, 3, 2, 3]
    check(inp, out, ref, max_band_frac=1.0)
    st = out.status.cpu().numpy()
    assert st.tolist() == [0, 5, 5, 0, 5, 0]
    # uniform p_n: the token is floor(u_k * V) wherever u_k * V is not within rounding of an integer
    tok = out.tokens.cpu().numpy()
    for b, n in [(1, 1), (2, 0), (4, 2)]:
        t = float(inp.uniforms[b, cfg.k]) * V
        if abs(t - round(t)) > 1e-3:
            assert tok[b, n] == int(t)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_row_without_finite_entries_sets_bad_row(binding, dtype):
    """A target or draft row of -inf only: the sequence carries SD_STATUS_BAD_ROW, its other outputs
    are unspecified but well-formed, and its neighbours are exact."""
    cfg = synth.custom_config(B=4, k=2, V=2048, dtype=dtype, index=67)
    inp = synth.make_inputs(cfg)
    ninf = np.float32(-np.inf) if dtype == "f32" else np.uint16(0xFF80)
    inp.target_logits[1, 0, :] = ninf
    inp.draft_logits[2, 1, :] = ninf
    T, D, x, u = to_device(inp)
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    ref = oracle_of(inp)
    assert ref.status.tolist() == [0, 2, 2, 0]
    st = out.status.cpu().numpy()
    assert st[0] == 0 and st[3] == 0 and (st[1] & binding.SD_STATUS_BAD_ROW) and (st[2] & binding.SD_STATUS_BAD_ROW)
    n = out.accept_len.cpu().numpy()
    tok = out.tokens.cpu().numpy()
    assert ((n >= 0) & (n <= cfg.k)).all()
    for b in range(cfg.B):
        assert 0 <= tok[b, n[b]] < cfg.V and (tok[b, n[b] + 1:] == -1).all()
    good = [0, 3]
    check(inp, out, oracle_of(inp, good), seqs=good, max_band_frac=1.0)


# ------------------------------------------------------------------ modes and plumbing
def test_library_scratch_survives_changing_batch_sizes_and_other_entry_points(binding):
    """The 13-argument entry point keeps one scratch buffer per device, and where the words that must
    start at zero end depends on the batch size: a small batch, then a larger one in the same
    buffer, then a smaller one, then after each of the other entry points that borrow the buffer.
    Every call must equal the call with a fresh caller workspace, bit for bit."""
    binding.sd_release_cached_buffers()
    k, V = 3, 8192

    def one(B, index):
        cfg = synth.custom_config(B=B, k=k, V=V, dtype="f32", index=index)
        inp = synth.make_inputs(cfg)
        T, D, x, u = to_device(inp)
        ref = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau, want_acc_prob=False, want_status=False)
        out = binding.sd_verify_feedback(T, D, x, u, inp.tau,
                                         out=binding.StepOutputs(accept_len=torch.full_like(ref.accept_len, -9),
                                                                 tokens=torch.full_like(ref.tokens, -9),
                                                                 loss=torch.full_like(ref.loss, -9.0),
                                                                 grad_draft=torch.full_like(ref.grad_draft, -9.0)))
        torch.cuda.synchronize()
        assert torch.equal(out.accept_len, ref.accept_len), f"B={B}: accept lengths"
        assert torch.equal(out.tokens, ref.tokens), f"B={B}: tokens"
        assert torch.equal(out.loss, ref.loss), f"B={B}: loss"
        assert torch.equal(out.grad_draft, ref.grad_draft), f"B={B}: gradient"
        return T, D, x, u, inp

    one(4, 80)
    one(200, 81)          # same buffer (under 1 MiB): the head of the layout is longer now
    one(70, 82)
    T, D, x, u, inp = one(130, 83)
    binding.sd_verify_error_feedback(T, D, x, u, inp.tau)          # borrows the library's buffer
    one(200, 84)
    one(5, 85)
    binding.sd_verify_greedy(T, x)
    one(190, 86)
    binding.sd_ensemble_feedback(T, [D, D], inp.tau, 10.0)
    one(66, 87)
    one(3, 88)
    binding.sd_verify_greedy(T, x)
    binding.sd_verify_greedy(T, x)
    torch.cuda.synchronize()



def test_verify_only_mode(binding):
    cfg = synth.custom_config(B=4, k=3, V=16000, dtype="bf16", index=61)
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)
    full = binding.sd_verify_feedback(T, D, x, u, inp.tau)
    only = binding.sd_verify_feedback(T, D, x, u, inp.tau, want_loss=False, want_grad=False)
    torch.cuda.synchronize()
    assert only.loss is None and only.grad_draft is None
    assert (full.accept_len == only.accept_len).all() and (full.tokens == only.tokens).all()


def test_results_are_deterministic(binding):
    cfg = synth.CONFIGS["cfg2"]
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)
    a = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    b = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    for name in ["accept_len", "tokens", "loss", "acc_prob", "status"]:
        assert torch.equal(getattr(a, name), getattr(b, name))
    assert torch.equal(a.grad_draft.view(torch.int16), b.grad_draft.view(torch.int16))


def test_dirty_workspace_and_guard_words(binding):
    """Caller scratch full of garbage is fine, and nothing is written outside the outputs."""
    cfg = synth.custom_config(B=5, k=3, V=12345 * 8, dtype="bf16", index=62)
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)
    B, k, V = cfg.B, cfg.k, cfg.V
    ws = torch.full((binding.sd_workspace_bytes(B, k, V, binding.SD_DTYPE_BF16),), 0xFF, dtype=torch.uint8, device="cuda")
    pad = 64

    def guarded(shape, dtype, fill):
        n = int(np.prod(shape))
        buf = torch.full((n + 2 * pad,), fill, dtype=dtype, device="cuda")
        return buf, buf[pad:pad + n].view(shape)

    bufs = {}
    bufs["n"], n_v = guarded((B,), torch.int32, -77)
    bufs["tok"], tok_v = guarded((B, k + 1), torch.int32, -77)
    bufs["loss"], loss_v = guarded((B, k), torch.float32, -77.0)
    bufs["grad"], grad_v = guarded((B, k, V), torch.bfloat16, -77.0)
    bufs["acc"], acc_v = guarded((B, k), torch.float32, -77.0)
    bufs["st"], st_v = guarded((B,), torch.int32, -77)
    out = binding.StepOutputs(accept_len=n_v, tokens=tok_v, loss=loss_v, grad_draft=grad_v, acc_prob=acc_v, status=st_v)
    binding.sd_verify_feedback_ex(T, D, x, u, inp.tau, workspace=ws, out=out)
    torch.cuda.synchronize()
    for name, buf in bufs.items():
        assert (buf[:pad].float() == -77).all() and (buf[-pad:].float() == -77).all(), f"{name} guard words touched"
    check(inp, out, oracle_of(inp), max_band_frac=1.0)


def test_non_default_stream_and_changing_shapes(binding):
    s = torch.cuda.Stream()
    for (B, k, V, dtype) in [(2, 2, 8000, "f32"), (6, 4, 64000, "bf16"), (1, 1, 8, "f32"), (3, 3, 33000, "f32")]:
        cfg = synth.custom_config(B=B, k=k, V=V, dtype=dtype, index=63)
        inp = synth.make_inputs(cfg)
        T, D, x, u = to_device(inp)
        torch.cuda.synchronize()
        with torch.cuda.stream(s):
            out = binding.sd_verify_feedback(T, D, x, u, inp.tau)
        s.synchronize()
        check(inp, out, oracle_of(inp), max_band_frac=1.0)


def test_a_wait_that_runs_out_is_reported_and_leaves_the_library_usable(binding, options):
    """Every wait inside the fast path is bounded.  With the bound set to a few polls (an option
    that exists for this purpose) the first wait for data gives up long before the data can be
    there: the kernel must come back on its own, flag the sequences with SD_STATUS_TIMEOUT, and
    the next call with the usual bound must be exact again.  Nothing is made to hang: the waits
    simply run out."""
    cfg = synth.custom_config(B=6, k=3, V=40000, dtype="f32", index=68)
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)
    options(binding.SD_OPT_WAIT_POLLS, 4)
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()                                  # the kernel returned
    assert binding.sd_launch_info()["path"] == 1
    st = out.status.cpu().numpy().astype(np.uint32)
    assert (st & np.uint32(binding.SD_STATUS_TIMEOUT)).all(), st
    # the error-position and ensemble entry points share the waits
    err = binding.sd_verify_error_feedback(T, D, x, u, inp.tau)
    ens = binding.sd_ensemble_feedback(T, [D, D], inp.tau, 10.0, want_status=True)
    torch.cuda.synchronize()
    assert (err.status.cpu().numpy().astype(np.uint32) & np.uint32(binding.SD_STATUS_TIMEOUT)).all()
    assert (ens.status.cpu().numpy().astype(np.uint32) & np.uint32(binding.SD_STATUS_TIMEOUT)).all()
    # back to the usual bound: exact again, on caller scratch and on the library's own
    options(binding.SD_OPT_WAIT_POLLS, 1 << 21)
    binding.sd_release_cached_buffers()
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    ref = oracle_of(inp)
    check(inp, out, ref, max_band_frac=1.0)
    out2 = binding.sd_verify_feedback(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    check(inp, out2, ref, max_band_frac=1.0)


@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_host_entry_point_matches_device_entry_point(binding, name):
    cfg = synth.CONFIGS[name]
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)
    dev = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    hT = torch.from_numpy(inp.target_logits)
    hD = torch.from_numpy(inp.draft_logits)
    if cfg.dtype == "bf16":
        hT, hD = hT.view(torch.bfloat16), hD.view(torch.bfloat16)
    host = binding.sd_verify_feedback_host(hT.pin_memory(), hD.pin_memory(), torch.from_numpy(inp.draft_tokens),
                                           torch.from_numpy(inp.uniforms), inp.tau, want_acc_prob=True,
                                           want_status=True)
    assert torch.equal(host.accept_len, dev.accept_len.cpu())
    assert torch.equal(host.tokens, dev.tokens.cpu())
    # the host entry point works in slices of sequences, which may pick another cluster size:
    # sums are then taken in another order, so floating-point outputs agree to rounding only
    torch.testing.assert_close(host.loss, dev.loss.cpu(), rtol=1e-5, atol=4e-7)
    torch.testing.assert_close(host.grad_draft.float(), dev.grad_draft.cpu().float(), rtol=1e-2, atol=1e-7)
    torch.testing.assert_close(host.acc_prob, dev.acc_prob.cpu(), rtol=0, atol=1e-6)
    assert torch.equal(host.status, dev.status.cpu())


def test_host_entry_point_slices_large_batches(binding):
    """More than one slice of sequences (the slices overlap copies and kernels)."""
    cfg = synth.CONFIGS["cfg5"].with_batch(40)   # ~0.39 GB of logits and gradient: five slices
    inp = synth.make_inputs(cfg)
    host = binding.sd_verify_feedback_host(torch.from_numpy(inp.target_logits), torch.from_numpy(inp.draft_logits),
                                           torch.from_numpy(inp.draft_tokens), torch.from_numpy(inp.uniforms), inp.tau)
    seqs = [0, 7, 8, 23, 39]
    ref = oracle_of(inp, seqs)
    check(inp, host, ref, seqs=seqs, max_band_frac=1.0)


@pytest.mark.parametrize("name", ["cfg3", "cfg4"])
def test_pinsker_ties_acceptance_probability_to_the_loss_on_every_row(binding, name):
    """TV(p,q) <= sqrt(KL(p||q)/2) (used in the proof of Lemma 1), with TV = 1 - acc_prob (Eq. 1):
    holds for every row of a full-size workload whatever the oracle says; also 0 <= acc_prob <= 1."""
    cfg = synth.CONFIGS[name]
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)
    out = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau, want_grad=False)
    torch.cuda.synchronize()
    acc = out.acc_prob.cpu().numpy().astype(np.float64)
    loss = out.loss.cpu().numpy().astype(np.float64)
    assert ((acc >= -1e-6) & (acc <= 1 + 1e-6)).all()
    assert ((1.0 - acc) <= np.sqrt(loss / 2.0) + 1e-5).all()
    assert (out.status.cpu().numpy() == 0).all()


# ------------------------------------------------------------------ hint error of the optimistic update
def hint_of(inp, seed):
    """A stand-in for the last round's gradient: this round's oracle gradient of other inputs, i.e. a
    tensor with the scale and structure of a gradient (rows that sum to zero, most mass on few entries)."""
    other = synth.make_inputs(inp.cfg, seed)
    ref = sd_oracle.verify_feedback(other.target_logits, other.draft_logits, other.draft_tokens, other.uniforms,
                                    other.tau, want_grad=True, nthreads=min(8, sd_oracle.max_threads()))
    g = ref.grad.astype(np.float32)
    return synth.f32_to_bf16_bits(g) if inp.cfg.dtype == "bf16" else g


def check_hint_error(inp, hint_bits, got, tol):
    want = sd_oracle.hint_error(inp.target_logits, inp.draft_logits, hint_bits, inp.tau)
    err = np.abs(got.astype(np.float64) - want)
    assert (err <= tol * want + 1e-12).all(), f"hint error: worst ratio {np.max(err / (tol * want + 1e-12)):.3g}"


@pytest.mark.parametrize("dtype,B,k,V", [("f32", 5, 3, 32000), ("bf16", 5, 3, 32000), ("f32", 20, 4, 128256),
                                         ("bf16", 33, 2, 151936), ("f32", 3, 2, 1001), ("bf16", 2, 1, 777)])
def test_hint_error_matches_the_oracle(binding, dtype, B, k, V):
    """Sec. 3.2: sum_v (h - grad)^2 per position, h a gradient-like tensor; every other output is the
    plain step's.  The difference is taken against the fp32 gradient before it is rounded to the output
    type, so bf16 logits cost no accuracy here: every entry of that gradient carries a relative error of
    a few 2^-22 of max(p,q)/tau, and the fp32 partial sums of a warp add about as much again.  Bars:
    2e-4 (fp32 logits) and 1e-3 (bf16 logits, whose hint is itself coarse) of the exact value."""
    cfg = synth.custom_config(B, k, V, dtype=dtype, tau=0.9, index=80)
    inp = synth.make_inputs(cfg)
    hint_bits = hint_of(inp, synth.BASE_SEED + 7)
    T, D, x, u = to_device(inp)
    H = torch.from_numpy(hint_bits).cuda()
    if dtype == "bf16":
        H = H.view(torch.bfloat16)
    out = binding.sd_verify_feedback_hint(T, D, x, u, inp.tau, H)
    torch.cuda.synchronize()
    ref = oracle_of(inp)
    check(inp, out, ref, max_band_frac=0.5)
    check_hint_error(inp, hint_bits, out.hint_err.cpu().numpy(), 2e-4 if dtype == "f32" else 1e-3)
    plain = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    assert torch.equal(plain.grad_draft.view(torch.uint8), out.grad_draft.view(torch.uint8))
    assert torch.equal(plain.tokens, out.tokens) and torch.equal(plain.loss, out.loss)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_hint_error_in_place_and_special_hints(binding, dtype):
    """The gradient may replace the hint in its own buffer; a hint equal to the gradient the step writes
    gives the rounding of the output type only (zero for fp32), a zero hint gives the gradient's norm."""
    cfg = synth.custom_config(6, 3, 50000, dtype=dtype, tau=1.1, index=81)
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)
    first = binding.sd_verify_feedback_ex(T, D, x, u, inp.tau)
    torch.cuda.synchronize()
    same = binding.sd_verify_feedback_hint(T, D, x, u, inp.tau, first.grad_draft)
    torch.cuda.synchronize()
    g = first.grad_draft.float().cpu().numpy().astype(np.float64)
    norm2 = (g * g).sum(-1)
    if dtype == "f32":
        assert (same.hint_err.cpu().numpy() == 0).all()
    else:
        assert (same.hint_err.cpu().numpy() <= 2.0 ** -16 * norm2).all()      # (2^-8 relative per entry)^2
    zero = binding.sd_verify_feedback_hint(T, D, x, u, inp.tau, torch.zeros_like(D))
    torch.cuda.synchronize()
    ref = oracle_of(inp)
    want = (ref.grad * ref.grad).sum(-1)
    assert np.abs(zero.hint_err.cpu().numpy() - want).max() <= 1e-4 * want.max()
    # in place: the hint's buffer receives the gradient
    hint_bits = hint_of(inp, synth.BASE_SEED + 9)
    H = torch.from_numpy(hint_bits).cuda()
    if dtype == "bf16":
        H = H.view(torch.bfloat16)
    inplace = binding.sd_verify_feedback_hint(T, D, x, u, inp.tau, H, grad_out=H)
    torch.cuda.synchronize()
    assert torch.equal(H.view(torch.uint8), first.grad_draft.view(torch.uint8))
    check_hint_error(inp, hint_bits, inplace.hint_err.cpu().numpy(), 2e-4 if dtype == "f32" else 1e-3)


def test_hint_error_every_cluster_size_and_the_generic_path(binding, options):
    cfg = synth.custom_config(7, 2, 65536, dtype="bf16", tau=0.8, index=82)
    inp = synth.make_inputs(cfg)
    hint_bits = hint_of(inp, synth.BASE_SEED + 11)
    T, D, x, u = to_device(inp)
    H = torch.from_numpy(hint_bits).cuda().view(torch.bfloat16)
    for cluster in (1, 2, 3, 5, 8):
        options(binding.SD_OPT_CLUSTER, cluster)
        out = binding.sd_verify_feedback_hint(T, D, x, u, inp.tau, H)
        torch.cuda.synchronize()
        assert binding.sd_launch_info()["cluster_size"] == cluster
        check_hint_error(inp, hint_bits, out.hint_err.cpu().numpy(), 1e-3)
    options(binding.SD_OPT_CLUSTER, 0)
    options(binding.SD_OPT_FORCE_GENERIC, 1)
    out = binding.sd_verify_feedback_hint(T, D, x, u, inp.tau, H)
    torch.cuda.synchronize()
    assert binding.sd_launch_info()["path"] == 0
    check_hint_error(inp, hint_bits, out.hint_err.cpu().numpy(), 1e-3)


def test_hint_entry_refusals(binding):
    cfg = synth.custom_config(2, 2, 4096, dtype="f32", index=83)
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)
    with pytest.raises(ValueError):
        binding.sd_verify_feedback_hint(T, D, x, u, inp.tau, torch.zeros((2, 2, 4000), device="cuda"))
    with pytest.raises(binding.SdVerifyError):
        binding.sd_verify_feedback_hint(T, D, x, u, inp.tau, torch.zeros_like(D),
                                        workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
