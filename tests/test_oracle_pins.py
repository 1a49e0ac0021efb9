"""Pins for the CPU oracle: everything it computes is checked against something that is not the
oracle -- hand-worked cases, closed forms, brute-force enumeration, finite differences and
library routines (scipy).  CPU only."""
import json
import math
import os

import numpy as np
import pytest
from scipy.special import logsumexp, rel_entr, softmax

from oracle import sd_oracle
from paper_2603_12617_b200 import synth

HERE = os.path.dirname(os.path.abspath(__file__))


def run(T, D, x, u, tau=1.0, **kw):
    T = np.asarray(T, np.float32)
    D = np.asarray(D, np.float32)
    if T.ndim == 2:
        T, D = T[None], D[None]
        x, u = np.asarray(x)[None], np.asarray(u)[None]
    return sd_oracle.verify_feedback(T, D, np.asarray(x, np.int32), np.asarray(u, np.float32), tau, **kw)


def logits_of(prob):
    return np.log(np.asarray(prob, np.float64)).astype(np.float32)


# ---------------------------------------------------------------- hand-worked cases (Algorithm 1)
with open(os.path.join(HERE, "golden", "hand_cases.json")) as fh:
    HAND = json.load(fh)["cases"]


@pytest.mark.parametrize("case", HAND, ids=[c["name"] for c in HAND])
def test_hand_cases(case):
    res = run(logits_of(case["p"]), logits_of(case["q"]), case["x"], case["u"])
    assert res.accept_len[0] == case["accept_len"]
    assert res.tokens[0].tolist() == case["tokens"]
    np.testing.assert_allclose(res.ratio[0], case["ratio"], rtol=1e-6)
    np.testing.assert_allclose(res.acc_prob[0], case["acc_prob"], rtol=1e-6)
    assert res.status[0] == 0


def test_residual_draw_every_uniform_two_token():
    # p=(1/2,1/2), q=(3/4,1/4): a rejection of token 0 must emit token 1 for every u_k
    uk = np.linspace(0, 1, 257, endpoint=False, dtype=np.float32)
    B = uk.size
    T = np.broadcast_to(logits_of([[0.5, 0.5], [0.5, 0.5]]), (B, 2, 2))
    D = np.broadcast_to(logits_of([[0.75, 0.25]]), (B, 1, 2))
    u = np.stack([np.full(B, 0.9, np.float32), uk], axis=1)
    res = run(T, D, np.zeros((B, 1)), u)
    assert (res.accept_len == 0).all() and (res.tokens[:, 0] == 1).all()


def test_inverse_cdf_edges():
    p = np.array([0.0625, 0.25, 0.1875, 0.5])  # dyadic: cumulative sums are exact
    T = logits_of([p, p])
    D = logits_of([p])
    # all accepted (p = q), bonus draw from p with u_k on either side of each edge
    edges = np.cumsum(p)[:-1]
    for j, e in enumerate(edges):
        below = np.nextafter(np.float32(e), np.float32(0)) - np.float32(1e-6)
        above = np.float32(e) + np.float32(1e-6)
        assert run(T, D, [0], [0.5, below]).tokens[0, 1] == j
        assert run(T, D, [0], [0.5, above]).tokens[0, 1] == j + 1
    assert run(T, D, [0], [0.5, 0.0]).tokens[0, 1] == 0
    assert run(T, D, [0], [0.5, np.nextafter(np.float32(1), np.float32(0))]).tokens[0, 1] == 3


def test_zero_mass_tokens_never_drawn():
    # residual (0, 0, 0.3, 0): u_k = 0 must skip the zero-mass tokens 0 and 1
    p = [0.2, 0.3, 0.45, 0.05]
    q = [0.45, 0.35, 0.15, 0.05]
    for uk in [0.0, 0.5, 0.999]:
        res = run(logits_of([p, p]), logits_of([q]), [0], [0.99, uk])
        assert res.accept_len[0] == 0 and res.tokens[0, 0] == 2


# ---------------------------------------------------------------- softmax (library routine)
@pytest.mark.parametrize("tau", [1.0, 0.6, 2.5])
def test_softmax_ratio_and_accprob_match_scipy(tau):
    rng = np.random.default_rng(1)
    V, k = 37, 3
    T = rng.normal(0, 3, (k + 1, V)).astype(np.float32)
    D = rng.normal(0, 3, (k, V)).astype(np.float32)
    p = softmax(T.astype(np.float64) / tau, axis=1)
    q = softmax(D.astype(np.float64) / tau, axis=1)
    x = rng.integers(0, V, k)
    res = run(T, D, x, rng.random(k + 1), tau)
    np.testing.assert_allclose(res.ratio[0], [p[i, x[i]] / q[i, x[i]] for i in range(k)], rtol=1e-12)
    np.testing.assert_allclose(res.acc_prob[0], np.minimum(p[:k], q).sum(1), rtol=1e-12)
    np.testing.assert_allclose(res.grad[0], (q - p[:k]) / tau, rtol=1e-10, atol=1e-15)


def test_shift_invariance_and_large_logits():
    rng = np.random.default_rng(2)
    V, k = 50, 2
    T = rng.normal(0, 2, (k + 1, V)).astype(np.float32)
    D = rng.normal(0, 2, (k, V)).astype(np.float32)
    x, u = rng.integers(0, V, k), rng.random(k + 1)
    # +64 / -80 are exactly representable shifts for these magnitudes up to fp32 rounding of the
    # sum, so use values on a coarse grid where the shifted logits stay exact
    Tq = np.round(T * 64) / 64
    Dq = np.round(D * 64) / 64
    a = run(Tq, Dq, x, u)
    b = run(Tq + np.float32(80.0), Dq - np.float32(80.0), x, u)
    assert (a.tokens == b.tokens).all()
    np.testing.assert_allclose(a.loss, b.loss, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(a.grad, b.grad, rtol=1e-12, atol=1e-16)
    np.testing.assert_allclose(a.ratio, b.ratio, rtol=1e-12)


# ---------------------------------------------------------------- Eq. 1: Acc = sum min(p,q) = 1 - TV
def test_acceptance_probability_identity():
    rng = np.random.default_rng(3)
    V = 8
    T = rng.normal(0, 1.5, (2, V)).astype(np.float32)
    D = rng.normal(0, 1.5, (1, V)).astype(np.float32)
    p = softmax(T[0].astype(np.float64))
    q = softmax(D[0].astype(np.float64))
    # E_{x~q} min(1, p/q) assembled from the oracle's ratio for each possible draft token
    ratios = np.array([run(T, D, [x], [0.5, 0.5]).ratio[0, 0] for x in range(V)])
    acc_from_ratio = float((q * np.minimum(1.0, ratios)).sum())
    acc_oracle = run(T, D, [0], [0.5, 0.5]).acc_prob[0, 0]
    tv = 0.5 * np.abs(p - q).sum()
    assert abs(acc_from_ratio - (1 - tv)) < 1e-12
    assert abs(acc_oracle - (1 - tv)) < 1e-12
    assert abs(acc_oracle - np.minimum(p, q).sum()) < 1e-12


def test_acceptance_frequency_monte_carlo():
    rng = np.random.default_rng(4)
    V, N = 6, 200000
    T = rng.normal(0, 1.0, (2, V)).astype(np.float32)
    D = rng.normal(0, 1.0, (1, V)).astype(np.float32)
    q = softmax(D[0].astype(np.float64))
    p = softmax(T[0].astype(np.float64))
    x = rng.choice(V, size=N, p=q)
    u = rng.random((N, 2)).astype(np.float32)
    res = run(np.broadcast_to(T, (N, 2, V)), np.broadcast_to(D, (N, 1, V)), x[:, None], u,
              want_grad=False)
    acc = np.minimum(p, q).sum()
    freq = (res.accept_len == 1).mean()
    assert abs(freq - acc) < 4 * math.sqrt(acc * (1 - acc) / N)


# ---------------------------------------------------------------- output marginal equals the target
def _marginal_by_grid(T, D, tau, n_accept, n_sample):
    """Emitted-token distribution per output position, conditional on the position being reached,
    by running the oracle on every draft-token tuple (weighted by q) and a midpoint grid of uniforms."""
    k, V = D.shape
    p = softmax(T.astype(np.float64) / tau, axis=1)
    q = softmax(D.astype(np.float64) / tau, axis=1)
    grids = [(np.arange(n_accept) + 0.5) / n_accept] * k + [(np.arange(n_sample) + 0.5) / n_sample]
    U = np.stack([g.ravel() for g in np.meshgrid(*grids, indexing="ij")], axis=1).astype(np.float32)
    N = U.shape[0]
    mass = np.zeros((k + 1, V))      # weight of emitting token y at output position j
    reach = np.zeros(k + 1)          # weight of reaching position j (first j drafts accepted)
    Tb = np.broadcast_to(T, (N, k + 1, V))
    Db = np.broadcast_to(D, (N, k, V))
    for xs in np.ndindex(*([V] * k)):
        w = np.prod([q[i, xs[i]] for i in range(k)]) / N
        res = run(Tb, Db, np.broadcast_to(np.array(xs), (N, k)), U, tau, want_grad=False, want_loss=False)
        for j in range(k + 1):
            reached = res.accept_len >= j
            reach[j] += w * reached.sum()
            # the token emitted at position j: draft token if accepted, the extra token if n == j
            emitted = res.tokens[reached, j]
            mass[j] += w * np.bincount(emitted, minlength=V)
    return mass / reach[:, None], p


def test_output_marginal_k1_fine_grid():
    rng = np.random.default_rng(5)
    V = 5
    T = rng.normal(0, 1.2, (2, V)).astype(np.float32)
    D = rng.normal(0, 1.2, (1, V)).astype(np.float32)
    marg, p = _marginal_by_grid(T, D, 1.0, n_accept=400, n_sample=400)
    assert np.abs(marg - p).max() < 5e-3 / 1  # midpoint grid: error <= 1/(2*400) per threshold


@pytest.mark.parametrize("k,V,tau", [(2, 4, 0.7), (3, 3, 1.3)])
def test_output_marginal_multi_position(k, V, tau):
    rng = np.random.default_rng(6 + k)
    T = rng.normal(0, 1.0, (k + 1, V)).astype(np.float32)
    D = rng.normal(0, 1.0, (k, V)).astype(np.float32)
    n = 40 if k == 2 else 16
    marg, p = _marginal_by_grid(T, D, tau, n_accept=n, n_sample=200)
    assert np.abs(marg - p).max() < 1.5 / n


def test_output_marginal_analytic_v8():
    # exact interval measure: P(out = y) = q_y min(1, p_y/q_y) + (1 - Acc) r_y / R must equal p_y,
    # with the ratio, acceptance probability and residual draw all taken from the oracle
    rng = np.random.default_rng(7)
    V = 8
    T = rng.normal(0, 1.5, (2, V)).astype(np.float32)
    D = rng.normal(0, 1.5, (1, V)).astype(np.float32)
    p = softmax(T[0].astype(np.float64))
    q = softmax(D[0].astype(np.float64))
    ratios = np.array([run(T, D, [x], [0.5, 0.5]).ratio[0, 0] for x in range(V)])
    # residual draw measured on a fine grid of u_k under a forced rejection (u_0 just below 1)
    M = 200000
    uk = ((np.arange(M) + 0.5) / M).astype(np.float32)
    x_rej = int(np.argmin(ratios))
    res = run(np.broadcast_to(T, (M, 2, V)), np.broadcast_to(D, (M, 1, V)), np.full((M, 1), x_rej),
              np.stack([np.full(M, 0.999999, np.float32), uk], 1), want_grad=False)
    assert (res.accept_len == 0).all()
    resid = np.bincount(res.tokens[:, 0], minlength=V) / M
    acc = res.acc_prob[0, 0]
    out = q * np.minimum(1.0, ratios) + (1 - acc) * resid
    assert np.abs(out - p).max() < 2e-5


# ---------------------------------------------------------------- expected accepted length (proof of Lemma 1)
def test_expected_emitted_tokens_closed_form():
    rng = np.random.default_rng(8)
    V, k, N = 7, 4, 100000
    t_row = rng.normal(0, 1.0, V).astype(np.float32)
    d_row = rng.normal(0, 1.0, V).astype(np.float32)
    p = softmax(t_row.astype(np.float64))
    q = softmax(d_row.astype(np.float64))
    acc = np.minimum(p, q).sum()
    T = np.broadcast_to(t_row, (N, k + 1, V))
    D = np.broadcast_to(d_row, (N, k, V))
    x = rng.choice(V, size=(N, k), p=q)
    res = run(T, D, x, rng.random((N, k + 1)), want_grad=False)
    emitted = res.accept_len + 1
    expect = (1 - acc ** (k + 1)) / (1 - acc)
    assert abs(emitted.mean() - expect) < 4 * emitted.std() / math.sqrt(N)


# ---------------------------------------------------------------- loss = KL(p||q) (Eq. kl_divergence)
@pytest.mark.parametrize("tau", [1.0, 0.8])
def test_loss_is_kl_scipy(tau):
    rng = np.random.default_rng(9)
    V, k = 300, 3
    T = rng.normal(0, 2, (k + 1, V)).astype(np.float32)
    D = rng.normal(0, 2, (k, V)).astype(np.float32)
    p = softmax(T.astype(np.float64) / tau, axis=1)[:k]
    q = softmax(D.astype(np.float64) / tau, axis=1)
    res = run(T, D, rng.integers(0, V, k), rng.random(k + 1), tau)
    np.testing.assert_allclose(res.loss[0], rel_entr(p, q).sum(1), rtol=1e-10)
    assert (res.loss >= 0).all()
    # Pinsker (proof of Lemma 1): TV <= sqrt(KL/2)
    assert ((1 - res.acc_prob) <= np.sqrt(res.loss / 2) + 1e-12).all()
    # cross-entropy form of Assumption 1: CE(p,q) = KL + H(p)
    ce = -(p * (D.astype(np.float64) / tau - logsumexp(D.astype(np.float64) / tau, axis=1, keepdims=True))).sum(1)
    ent = -(p * np.log(p)).sum(1)
    np.testing.assert_allclose(res.loss[0], ce - ent, rtol=1e-9)


def test_loss_two_token_closed_form():
    a, b = 0.3, 0.6
    res = run(logits_of([[a, 1 - a], [a, 1 - a]]), logits_of([[b, 1 - b]]), [0], [0.5, 0.5])
    kl = a * math.log(a / b) + (1 - a) * math.log((1 - a) / (1 - b))
    assert abs(res.loss[0, 0] - kl) < 1e-7  # fp32 logits of log(prob)


def test_identical_models_accept_everything():
    rng = np.random.default_rng(10)
    V, k, B = 1000, 5, 3
    T = (np.round(rng.normal(0, 3, (B, k + 1, V)) * 64) / 64).astype(np.float32)  # +4 stays exact
    D = T[:, :k].copy()
    x = rng.integers(0, V, (B, k))
    u = rng.random((B, k + 1)).astype(np.float32)
    res = run(T, D, x, u)
    assert (res.accept_len == k).all()
    assert (res.tokens[:, :k] == x).all() and (res.tokens[:, k] >= 0).all()
    assert np.abs(res.loss).max() == 0.0 and np.abs(res.grad).max() == 0.0
    np.testing.assert_allclose(res.acc_prob, 1.0, rtol=1e-12)
    # a constant shift of the draft logits changes nothing (softmax shift invariance)
    res2 = run(T, D + np.float32(4.0), x, u)
    assert (res2.accept_len == k).all()
    assert np.abs(res2.loss).max() < 1e-12 and np.abs(res2.grad).max() < 1e-12


# ---------------------------------------------------------------- gradient: finite differences
@pytest.mark.parametrize("tau", [1.0, 0.6, 1.7])
def test_gradient_finite_differences(tau):
    rng = np.random.default_rng(11)
    V, k = 12, 2
    T = rng.normal(0, 1.5, (k + 1, V))
    D = rng.normal(0, 1.5, (k, V))

    def loss_of(Dm):
        # fp32 logits cannot carry an h = 1e-3 perturbation cleanly: scale so values are exact
        return run(T.astype(np.float32), Dm.astype(np.float32), [0] * k, [0.5] * (k + 1), tau,
                   want_grad=False).loss[0]

    # use a grid of exactly representable logits and a power-of-two step
    T = np.round(T * 256) / 256
    D = np.round(D * 256) / 256
    h = 2.0 ** -9
    g = run(T.astype(np.float32), D.astype(np.float32), [0] * k, [0.5] * (k + 1), tau).grad[0]
    assert np.abs(g.sum(1)).max() < 1e-12
    for i in range(k):
        for v in range(V):
            Dp, Dm = D.copy(), D.copy()
            Dp[i, v] += h
            Dm[i, v] -= h
            fd = (loss_of(Dp)[i] - loss_of(Dm)[i]) / (2 * h)
            # central differences: error O(h^2 * third derivative) ~ 4e-6 / tau^3
            assert abs(fd - g[i, v]) < 2e-5 / tau ** 3, (i, v, fd, g[i, v])
            # the loss of the other position does not move
            j = 1 - i
            assert loss_of(Dp)[j] == loss_of(Dm)[j]


# ---------------------------------------------------------------- data handling
def test_bf16_logits_are_widened_exactly():
    cfg = synth.custom_config(B=2, k=3, V=257, dtype="bf16", tau=0.9)
    inp = synth.make_inputs(cfg)
    a = sd_oracle.verify_feedback(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, inp.tau)
    b = sd_oracle.verify_feedback(synth.bf16_bits_to_f32(inp.target_logits),
                                  synth.bf16_bits_to_f32(inp.draft_logits), inp.draft_tokens,
                                  inp.uniforms, inp.tau)
    assert (a.tokens == b.tokens).all() and (a.loss == b.loss).all() and (a.grad == b.grad).all()


def test_sequences_are_independent_and_threads_do_not_change_results():
    cfg = synth.custom_config(B=6, k=3, V=401, dtype="f32", tau=1.1)
    inp = synth.make_inputs(cfg)
    args = (inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, inp.tau)
    full = sd_oracle.verify_feedback(*args, nthreads=1)
    par = sd_oracle.verify_feedback(*args, nthreads=4)
    for name in ["accept_len", "tokens", "loss", "grad", "acc_prob", "ratio", "cdf_margin"]:
        assert (getattr(full, name) == getattr(par, name)).all()
    for b in range(cfg.B):
        one = sd_oracle.verify_feedback(*(a[b:b + 1] for a in args[:4]), inp.tau)
        assert (one.tokens[0] == full.tokens[b]).all() and (one.loss[0] == full.loss[b]).all()


def test_masked_vocabulary_entries():
    rng = np.random.default_rng(12)
    V, k = 20, 2
    T = rng.normal(0, 1, (k + 1, V)).astype(np.float32)
    D = rng.normal(0, 1, (k, V)).astype(np.float32)
    T[:, 3] = -np.inf           # target never emits token 3
    p = softmax(T.astype(np.float64), axis=1)
    q = softmax(D.astype(np.float64), axis=1)
    res = run(T, D, [3, 5], [0.0, 0.5, 0.5])
    assert res.ratio[0, 0] == 0.0 and res.accept_len[0] == 0   # p(3) = 0: rejected even at u = 0
    assert res.tokens[0, 0] != 3
    np.testing.assert_allclose(res.loss[0], rel_entr(p[:k], q).sum(1), rtol=1e-10)
    np.testing.assert_allclose(res.grad[0, :, 3], q[:, 3], rtol=1e-10)
    D2 = D.copy()
    D2[0, 7] = -np.inf          # draft gives zero mass where the target does not: infinite KL
    assert np.isinf(run(T, D2, [1, 1], [0.5, 0.5, 0.5]).loss[0, 0])


def test_bad_token_sets_status_and_rejects():
    rng = np.random.default_rng(13)
    V, k = 9, 3
    T = rng.normal(0, 1, (k + 1, V)).astype(np.float32)
    res = run(T, T[:k], [1, V, 2], [0.1, 0.1, 0.1, 0.1])
    assert res.status[0] & 1 and res.accept_len[0] == 1 and res.tokens[0, 0] == 1


def test_zero_residual_at_a_forced_rejection_draws_from_p():
    """A rejection whose residual max(0, p - q) has no mass (only a token outside the vocabulary can
    force one when q = p): the extra token comes from p_n by the same inverse CDF, and the status
    says so.  Edges of p at 1/16, 5/16, 1/2, 1; the uniforms stay clear of them."""
    p = np.array([0.0625, 0.25, 0.1875, 0.5])
    V = p.size
    T = logits_of([p, p, p])
    D = logits_of([p, p])
    for uk, want in [(0.0, 0), (0.06, 0), (0.07, 1), (0.3, 1), (0.4, 2), (0.51, 3), (0.999, 3)]:
        res = run(T, D, [1, V], [0.99, 0.0, uk])          # ratio 1 accepts whatever u_0 is; token V is no token
        assert res.accept_len[0] == 1 and res.tokens[0].tolist() == [1, want, -1]
        assert res.status[0] == 1 | 4                      # BAD_TOKEN | ZERO_RESIDUAL
        assert res.ratio[0, 1] == 0.0
    # a negative token at position 0, and a residual with mass elsewhere in the batch is untouched
    res = run(T, D, [-1, 2], [0.0, 0.0, 0.3])
    assert res.accept_len[0] == 0 and res.tokens[0].tolist() == [1, -1, -1] and res.status[0] == 5
    # the same forced rejection with q != p has a residual: no fallback, no flag 4
    q = np.array([0.25, 0.25, 0.25, 0.25])
    res = run(T, logits_of([q, q]), [V, 0], [0.5, 0.5, 0.5])   # residual (0,0,0,1/4): token 3
    assert res.accept_len[0] == 0 and res.tokens[0, 0] == 3 and res.status[0] == 1


def test_row_without_a_softmax_denominator_sets_bad_row():
    """A row of -inf only has no finite positive denominator: the sequence is flagged (its outputs
    are unspecified), its neighbours are not."""
    rng = np.random.default_rng(14)
    V, k = 6, 2
    T = rng.normal(0, 1, (3, k + 1, V)).astype(np.float32)
    D = rng.normal(0, 1, (3, k, V)).astype(np.float32)
    T[1, 0, :] = -np.inf                                   # a target row
    D[2, 1, :] = -np.inf                                   # a draft row
    x = np.zeros((3, k), np.int32)
    u = np.full((3, k + 1), 0.5, np.float32)
    res = sd_oracle.verify_feedback(T, D, x, u, 1.0)
    assert res.status.tolist() == [0, 2, 2]
    assert (res.accept_len >= 0).all() and (res.accept_len <= k).all()


def test_draw_interval_hand_values_and_agreement_with_the_draw():
    """p = (.1,.2,.3,.4), q = (.4,.3,.2,.1): residual (0,0,.1,.3), R = .4, so token 2 owns [0,.1) and
    token 3 owns [.1,.4); tokens 0 and 1 own empty intervals.  Bonus position: the edges of p."""
    p = [0.1, 0.2, 0.3, 0.4]
    q = [0.4, 0.3, 0.2, 0.1]
    T = logits_of([p, p])
    D = logits_of([q])
    want = {0: (0.0, 0.0), 1: (0.0, 0.0), 2: (0.0, 0.1), 3: (0.1, 0.4)}
    for y, (lo, hi) in want.items():
        a, b, R = sd_oracle.draw_interval(T, D, 1.0, 0, y)
        np.testing.assert_allclose([a, b, R], [lo, hi, 0.4], atol=1e-7)
    edges = np.concatenate([[0.0], np.cumsum(p)])
    for y in range(4):
        a, b, R = sd_oracle.draw_interval(T, D, 1.0, 1, y)
        np.testing.assert_allclose([a, b, R], [edges[y], edges[y + 1], 1.0], atol=1e-7)
    # zero residual: the intervals of p_n
    a, b, R = sd_oracle.draw_interval(T, logits_of([p]), 1.0, 0, 2)
    np.testing.assert_allclose([a, b, R], [0.3, 0.6, 1.0], atol=1e-7)
    # whatever token sd_oracle draws, u_k * R lies in that token's interval
    rng = np.random.default_rng(15)
    k, V = 3, 23
    for trial in range(40):
        Tq = rng.normal(0, 2, (k + 1, V)).astype(np.float32)
        Dq = (Tq[:k] + rng.normal(0, 1, (k, V))).astype(np.float32)
        xs = rng.integers(0, V, k)
        us = rng.random(k + 1).astype(np.float32)
        res = run(Tq, Dq, xs, us, 0.8)
        n = int(res.accept_len[0])
        a, b, R = sd_oracle.draw_interval(Tq, Dq, 0.8, n, int(res.tokens[0, n]))
        assert a <= float(us[k]) * R < b


def test_accept_band_flag():
    p = [[0.5, 0.5], [0.5, 0.5]]
    q = [[0.75, 0.25]]
    rho = run(logits_of(p), logits_of(q), [0], [0.5, 0.5]).ratio[0, 0]
    near = np.float32(rho + 3e-7)
    far = np.float32(rho + 1e-4)
    assert run(logits_of(p), logits_of(q), [0], [near, 0.5]).accept_band[0, 0] == 1
    assert run(logits_of(p), logits_of(q), [0], [far, 0.5]).accept_band[0, 0] == 0
    # tests after the first rejection are never reached and never flagged
    T = logits_of([[0.5, 0.5], [0.5, 0.5], [0.5, 0.5]])
    D = logits_of([[0.75, 0.25], [0.75, 0.25]])
    res = run(T, D, [0, 0], [0.9, near, 0.5])
    assert res.accept_len[0] == 0 and res.accept_band[0].tolist() == [0, 0]


def test_cdf_margin():
    p = np.array([0.25, 0.25, 0.5])
    T, D = logits_of([p, p]), logits_of([p])
    res = run(T, D, [0], [0.5, 0.3])          # bonus draw: t = 0.3 in [0.25, 0.5): margin 0.05
    assert res.tokens[0, 1] == 1 and abs(res.cdf_margin[0] - 0.05) < 1e-6


# ---------------------------------------------------------------- greedy verification (tau -> 0)
def test_greedy_hand_cases():
    # rows: argmax 2, 0 (tie between 0 and 3: first index), 1
    T = np.array([[[0.1, 0.5, 2.0, -1.0], [3.0, 1.0, 0.0, 3.0], [-2.0, 7.5, 7.25, 0.0]]], np.float32)
    r = sd_oracle.verify_greedy(T, np.array([[2, 0]], np.int32))
    assert r.argmax.tolist() == [[2, 0, 1]] and r.accept_len.tolist() == [2] and r.tokens.tolist() == [[2, 0, 1]]
    r = sd_oracle.verify_greedy(T, np.array([[2, 3]], np.int32))      # 3 ties with 0 but is not the first index
    assert r.accept_len.tolist() == [1] and r.tokens.tolist() == [[2, 0, -1]]
    r = sd_oracle.verify_greedy(T, np.array([[1, 0]], np.int32))
    assert r.accept_len.tolist() == [0] and r.tokens.tolist() == [[2, -1, -1]]


def test_greedy_argmax_matches_numpy_and_masks():
    rng = np.random.default_rng(21)
    B, k, V = 5, 3, 777
    T = rng.normal(0, 3, (B, k + 1, V)).astype(np.float32)
    T[0, 0, :] = -np.inf                       # nothing above -inf: index 0
    T[1, 2, 100:] = -np.inf
    T[2, 1, 5] = T[2, 1].max() + 1             # ties elsewhere do not matter
    x = rng.integers(0, V, (B, k)).astype(np.int32)
    r = sd_oracle.verify_greedy(T, x)
    assert (r.argmax == T.argmax(axis=2)).all()        # numpy's argmax also returns the first maximum
    bits = synth.f32_to_bf16_bits(T)
    rb = sd_oracle.verify_greedy(bits, x)
    assert (rb.argmax == synth.bf16_bits_to_f32(bits).argmax(axis=2)).all()


def test_greedy_is_the_small_temperature_limit_of_the_sampling_step():
    """With draft tokens decoded greedily from the draft, Algorithm 1 at a very small temperature
    accepts exactly the tokens that are the target's argmax and emits the target's argmax at the
    first mismatch, whatever the uniforms: the greedy oracle must agree with the sampling oracle."""
    rng = np.random.default_rng(22)
    B, k, V = 12, 4, 50
    T = rng.normal(0, 2, (B, k + 1, V)).astype(np.float32)
    D = (T[:, :k] + rng.normal(0, 1.0, (B, k, V))).astype(np.float32)
    x = D.argmax(axis=2).astype(np.int32)
    u = rng.random((B, k + 1)).astype(np.float32)
    # gaps between the two largest logits are ~0.1 .. 1 here; tau = 1e-3 makes the softmax a point mass
    samp = sd_oracle.verify_feedback(T, D, x, u, 1e-3, want_grad=False, want_loss=False)
    gr = sd_oracle.verify_greedy(T, x)
    assert (samp.accept_len == gr.accept_len).all()
    assert (samp.tokens == gr.tokens).all()
    assert len(set(gr.accept_len.tolist())) > 1       # the case exercises several accept lengths


# ---- online ensemble (Sec. 3.3): per-learner feedback and the Hedge weights ----------------

def _ensemble_case(seed=0, N=3, B=3, k=2, V=11):
    rng = np.random.default_rng(seed)
    T = rng.standard_normal((B, k + 1, V)).astype(np.float32) * 2.0
    Ds = [(T[:, :k] + (0.3 * 2 ** n) * rng.standard_normal((B, k, V))).astype(np.float32) for n in range(N)]
    return T, Ds


@pytest.mark.parametrize("tau", [0.6, 1.0])
def test_ensemble_losses_and_gradients_match_scipy_per_learner(tau):
    T, Ds = _ensemble_case(1)
    res = sd_oracle.ensemble_feedback(T, Ds, tau, eps=10.0)
    p = softmax(T[:, :-1].astype(np.float64) / tau, axis=-1)
    for n, D in enumerate(Ds):
        q = softmax(D.astype(np.float64) / tau, axis=-1)
        np.testing.assert_allclose(res.loss[n], rel_entr(p, q).sum(-1), rtol=1e-11, atol=1e-14)
        np.testing.assert_allclose(res.grad[n], (q - p) / tau, rtol=1e-11, atol=1e-15)
        assert res.round_loss[n] == pytest.approx(rel_entr(p, q).sum(-1).mean(), rel=1e-12)


def test_hedge_weights_hand_values():
    """Two learners with cumulative losses 0.1 and 0.2 and eps = 10: the weights are
    1/(1+e^-1) and e^-1/(1+e^-1) (the two-expert form of the exponential weighting scheme)."""
    T, Ds = _ensemble_case(2, N=2)
    Ds = [T[:, :-1].copy(), T[:, :-1].copy()]            # both learners equal the target: the round adds nothing
    res = sd_oracle.ensemble_feedback(T, Ds, 1.0, eps=10.0, cum_loss=np.array([0.1, 0.2]))
    np.testing.assert_allclose(res.round_loss, 0.0, atol=1e-15)
    np.testing.assert_allclose(res.cum_loss, [0.1, 0.2], rtol=1e-15)
    np.testing.assert_allclose(res.weights, [0.7310585786300049, 0.2689414213699951], rtol=1e-12)


def test_hedge_weights_are_softmax_of_minus_eps_cumulative_loss_and_accumulate_over_rounds():
    T, Ds = _ensemble_case(3)
    eps = 10.0
    cum = None
    total = np.zeros(3)
    for rnd in range(3):
        T, Ds = _ensemble_case(10 + rnd)
        res = sd_oracle.ensemble_feedback(T, Ds, 0.8, eps=eps, cum_loss=cum, want_grad=False)
        total += res.round_loss
        np.testing.assert_allclose(res.cum_loss, total, rtol=1e-13)
        np.testing.assert_allclose(res.weights, softmax(-eps * total), rtol=1e-12)
        assert res.weights.sum() == pytest.approx(1.0, abs=1e-15)
        cum = res.cum_loss
    # the noisier the learner the larger its loss, hence the smaller its weight
    assert res.weights[0] > res.weights[1] > res.weights[2]


def test_hedge_limits_and_invariance():
    T, Ds = _ensemble_case(4)
    base = sd_oracle.ensemble_feedback(T, Ds, 1.0, eps=10.0, cum_loss=np.array([0.3, 0.1, 0.2]), want_grad=False)
    # eps = 0: uniform weights, whatever the losses
    flat = sd_oracle.ensemble_feedback(T, Ds, 1.0, eps=0.0, cum_loss=np.array([0.3, 0.1, 0.2]), want_grad=False)
    np.testing.assert_allclose(flat.weights, 1.0 / 3.0, rtol=1e-15)
    # a constant added to every learner's cumulative loss (cross-entropy instead of KL: + entropy of p) cancels
    moved = sd_oracle.ensemble_feedback(T, Ds, 1.0, eps=10.0, cum_loss=np.array([0.3, 0.1, 0.2]) + 123.0, want_grad=False)
    np.testing.assert_allclose(moved.weights, base.weights, rtol=1e-10)
    # a huge eps puts all weight on the learner with the smallest cumulative loss, without overflow
    sharp = sd_oracle.ensemble_feedback(T, Ds, 1.0, eps=1e6, cum_loss=np.array([0.3, 0.1, 0.2]) * 1e3, want_grad=False)
    assert np.isfinite(sharp.weights).all()
    assert sharp.weights[int(np.argmin(sharp.cum_loss))] == pytest.approx(1.0)


def test_ensemble_learner_equals_single_draft_feedback_and_bf16():
    """Each learner's loss and gradient are those of the single-draft step given the same logits."""
    rng = np.random.default_rng(5)
    B, k, V = 2, 3, 37
    T = synth.f32_to_bf16_bits(rng.standard_normal((B, k + 1, V)).astype(np.float32) * 3)
    Ds = [synth.f32_to_bf16_bits(rng.standard_normal((B, k, V)).astype(np.float32) * 3) for _ in range(2)]
    res = sd_oracle.ensemble_feedback(T, Ds, 0.7, eps=10.0, nthreads=2)
    x = np.zeros((B, k), np.int32)
    u = np.zeros((B, k + 1), np.float32)
    for n in range(2):
        one = sd_oracle.verify_feedback(T, Ds[n], x, u, 0.7)
        np.testing.assert_allclose(res.loss[n], one.loss, rtol=1e-13)
        np.testing.assert_allclose(res.grad[n], one.grad, rtol=1e-13, atol=1e-300)


# ---- error-position feedback (what OSD collects, Sec. 3.1) ---------------------------------

def test_error_position_feedback_hand_cases():
    """Two-token vocabulary, tau = 1, logits = log-probabilities.  Sequence 0: p = (1/2,1/2),
    q = (3/4,1/4), x = 0, u = 0.7 > 2/3 rejects at position 0: the gradient row is q - p =
    (1/4,-1/4).  Sequence 1: the same pair accepted (u = 0.1), then q = (1/4,3/4) with x = 1 and
    ratio 2/3 rejected (u = 0.9): the row of position 1, (-1/4, 1/4).  Sequence 2: everything
    accepted: a zero row."""
    lp = lambda *a: np.log(np.array(a, np.float64))
    T = np.empty((3, 3, 2), np.float32)
    D = np.empty((3, 2, 2), np.float32)
    T[:] = lp(0.5, 0.5)
    D[0] = [lp(0.75, 0.25), lp(0.75, 0.25)]
    D[1] = [lp(0.75, 0.25), lp(0.25, 0.75)]
    D[2] = [lp(0.75, 0.25), lp(0.25, 0.75)]
    x = np.array([[0, 0], [0, 1], [0, 1]], np.int32)
    u = np.array([[0.7, 0.0, 0.3], [0.1, 0.9, 0.3], [0.1, 0.2, 0.3]], np.float32)
    res = sd_oracle.error_position_feedback(T, D, x, u, 1.0)
    assert list(res.full.accept_len) == [0, 1, 2]
    np.testing.assert_allclose(res.error_grad, [[0.25, -0.25], [-0.25, 0.25], [0.0, 0.0]], atol=1e-7)
    # a later rejection does not move the error position: sequence 0 would also reject at position 1 (u = 0.0 accepts; make it reject)
    u2 = u.copy(); u2[0, 1] = 0.99
    res2 = sd_oracle.error_position_feedback(T, D, x, u2, 1.0)
    np.testing.assert_allclose(res2.error_grad[0], [0.25, -0.25], atol=1e-7)


def test_error_position_feedback_is_a_selection_of_the_full_step():
    cfg = synth.custom_config(6, 4, 257, dtype="bf16", tau=0.7, recipe="peaks")
    inp = synth.make_inputs(cfg)
    res = sd_oracle.error_position_feedback(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, inp.tau)
    full = sd_oracle.verify_feedback(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, inp.tau)
    assert (res.full.tokens == full.tokens).all()
    for b in range(cfg.B):
        n = int(full.accept_len[b])
        expect = full.grad[b, n] if n < cfg.k else np.zeros(cfg.V)
        assert (res.error_grad[b] == expect).all()
        if n < cfg.k:
            assert abs(res.error_grad[b].sum()) < 1e-12          # a difference of two distributions


# ---- the step after the feedback: hint error (Sec. 3.2) and the output layer's gradient (Sec. 3.1) ----

def test_hint_error_hand_values():
    """p = (1/2,1/2), q = (3/4,1/4), tau = 1: the gradient is q - p = (1/4,-1/4).  Against the hint
    (1/2, 0) the squared distance is 1/16 + 1/16; against the gradient itself it is 0; at tau = 1/2
    the gradient doubles."""
    T = logits_of([[[0.5, 0.5], [0.5, 0.5]]])
    D = logits_of([[[0.75, 0.25]]])
    hint = np.array([[[0.5, 0.0]]], np.float32)
    np.testing.assert_allclose(sd_oracle.hint_error(T, D, hint, 1.0), [[0.125]], rtol=1e-6)
    np.testing.assert_allclose(sd_oracle.hint_error(T, D, np.array([[[0.25, -0.25]]], np.float32), 1.0), [[0.0]], atol=1e-14)
    # tau = 1/2 squares the probabilities before normalising: p stays (1/2,1/2), q = (9/10,1/10); g = 2 (q - p)
    np.testing.assert_allclose(sd_oracle.hint_error(T, D, np.zeros((1, 1, 2), np.float32), 0.5), [[2 * 0.8 ** 2]], rtol=1e-6)


def test_hint_error_is_the_squared_distance_to_the_oracles_gradient():
    rng = np.random.default_rng(31)
    B, k, V = 3, 2, 41
    T = rng.normal(0, 2, (B, k + 1, V)).astype(np.float32)
    D = (T[:, :k] + rng.normal(0, 1, (B, k, V))).astype(np.float32)
    hint = rng.normal(0, 0.05, (B, k, V)).astype(np.float32)
    tau = 0.8
    p = softmax(T[:, :k].astype(np.float64) / tau, axis=-1)
    q = softmax(D.astype(np.float64) / tau, axis=-1)
    want = ((hint.astype(np.float64) - (q - p) / tau) ** 2).sum(-1)
    np.testing.assert_allclose(sd_oracle.hint_error(T, D, hint, tau), want, rtol=1e-11)
    # bf16 inputs are widened exactly
    Tb, Db, hb = (synth.f32_to_bf16_bits(a) for a in (T, D, hint))
    p = softmax(synth.bf16_bits_to_f32(Tb)[:, :k].astype(np.float64) / tau, axis=-1)
    q = softmax(synth.bf16_bits_to_f32(Db).astype(np.float64) / tau, axis=-1)
    want = ((synth.bf16_bits_to_f32(hb).astype(np.float64) - (q - p) / tau) ** 2).sum(-1)
    np.testing.assert_allclose(sd_oracle.hint_error(Tb, Db, hb, tau), want, rtol=1e-11)


def test_lmhead_gradient_hand_case_and_numpy():
    """R = 2 positions, V = 2, d = 2: g = [[1,2],[3,4]], X = [[5,6],[7,8]]:
    dW = g^T X = [[1*5+3*7, 1*6+3*8], [2*5+4*7, 2*6+4*8]] = [[26,30],[38,44]]."""
    g = np.array([[1, 2], [3, 4]], np.float32)
    X = np.array([[5, 6], [7, 8]], np.float32)
    np.testing.assert_array_equal(sd_oracle.lmhead_grad(g, X), [[26, 30], [38, 44]])
    # not the transposed product, and not X^T g
    assert not np.array_equal(sd_oracle.lmhead_grad(g, X), g @ X)
    rng = np.random.default_rng(32)
    g = rng.normal(0, 1, (7, 13)).astype(np.float32)
    X = rng.normal(0, 1, (7, 5)).astype(np.float32)
    full = sd_oracle.lmhead_grad(g, X)
    np.testing.assert_allclose(full, g.astype(np.float64).T @ X.astype(np.float64), rtol=1e-12, atol=1e-14)
    # sampled entries equal the full result; linear in X
    vs, js = np.array([0, 12, 5, 5]), np.array([4, 0, 2, 3])
    np.testing.assert_array_equal(sd_oracle.lmhead_grad(g, X, vs, js), full[vs, js])
    np.testing.assert_allclose(sd_oracle.lmhead_grad(g, (2 * X).astype(np.float32)), 2 * full, rtol=1e-12)
    # bf16 operands are widened exactly
    gb, Xb = synth.f32_to_bf16_bits(g), synth.f32_to_bf16_bits(X)
    want = synth.bf16_bits_to_f32(gb).astype(np.float64).T @ synth.bf16_bits_to_f32(Xb).astype(np.float64)
    np.testing.assert_allclose(sd_oracle.lmhead_grad(gb, Xb), want, rtol=1e-12, atol=1e-14)


def test_lmhead_gradient_is_the_derivative_of_the_loss_in_the_output_layers_weights():
    """Draft logits D = X W^T for a small linear output layer: central finite differences of the
    oracle's summed loss in every entry of W equal g^T X with the oracle's own gradient g."""
    rng = np.random.default_rng(33)
    B, k, V, d = 2, 2, 6, 3
    tau = 0.9
    T = rng.normal(0, 1.5, (B, k + 1, V)).astype(np.float32)
    X = rng.normal(0, 1, (B * k, d))
    W = rng.normal(0, 1, (V, d))
    x = np.zeros((B, k), np.int32)
    u = np.zeros((B, k + 1), np.float32)

    def loss_of(Wm):
        # the oracle takes float32 logits: keep the perturbation visible by working at a coarse step
        D = (X @ Wm.T).reshape(B, k, V)
        Tq = T.astype(np.float64)
        p = softmax(Tq[:, :k] / tau, axis=-1)
        q = softmax(D / tau, axis=-1)
        return rel_entr(p, q).sum()

    D32 = (X @ W.T).reshape(B, k, V).astype(np.float32)
    res = sd_oracle.verify_feedback(T, D32, x, u, tau)
    # the oracle's loss is the KL that loss_of restates with scipy (pinned elsewhere); its gradient feeds g^T X
    dW = sd_oracle.lmhead_grad(res.grad.reshape(B * k, V).astype(np.float32), X.astype(np.float32))
    h = 1e-5
    fd = np.zeros_like(W)
    for v in range(V):
        for j in range(d):
            Wp, Wm = W.copy(), W.copy()
            Wp[v, j] += h
            Wm[v, j] -= h
            fd[v, j] = (loss_of(Wp) - loss_of(Wm)) / (2 * h)
    np.testing.assert_allclose(dW, fd, rtol=2e-4, atol=2e-6)      # float32 logits and operands
