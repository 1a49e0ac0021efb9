"""GPU parity of greedy verification (Algorithm 1 in the limit tau -> 0) against the CPU oracle.

Everything here is integer work decided by comparisons of the stored logits, so the bar is
bit-exact: accept lengths, emitted tokens and the argmax of every target row.
"""
import numpy as np
import pytest
import torch

from oracle import sd_oracle
from paper_2603_12617_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    import __graft_entry__ as entry
    entry.build()
    from paper_2603_12617_b200 import binding as b
    return b


def device_logits(T):
    t = torch.from_numpy(T).cuda()
    return t.view(torch.bfloat16) if T.dtype == np.uint16 else t


def planted_tokens(T, seed):
    """Draft tokens that agree with the target's argmax on a seeded prefix of every sequence, differ
    right after it, and are a coin flip between the argmax and something else behind the mismatch
    (a match behind the first mismatch must not count)."""
    B, k1, V = T.shape
    k = k1 - 1
    Tf = synth.bf16_bits_to_f32(T) if T.dtype == np.uint16 else T
    am = Tf.argmax(axis=-1).astype(np.int32)            # input construction only; the oracle has its own
    rng = np.random.default_rng(seed)
    n = rng.integers(0, k + 1, size=B)
    x = am[:, :k].copy()
    for b in range(B):
        if n[b] < k and V > 1:
            x[b, n[b]] = (am[b, n[b]] + 1 + rng.integers(0, V - 1)) % V
            for i in range(n[b] + 1, k):
                if rng.random() < 0.5:
                    x[b, i] = rng.integers(0, V)
    return x, n.astype(np.int32)


def run_and_compare(binding, T, x, **kw):
    ref = sd_oracle.verify_greedy(T, x)
    out = binding.sd_verify_greedy(device_logits(T), torch.from_numpy(x).cuda(), **kw)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(out.accept_len.cpu().numpy(), ref.accept_len)
    np.testing.assert_array_equal(out.tokens.cpu().numpy(), ref.tokens)
    if out.argmax is not None:
        np.testing.assert_array_equal(out.argmax.cpu().numpy(), ref.argmax)
    return ref


@pytest.mark.parametrize("name,seqs", [("cfg1", None), ("cfg2", None), ("cfg3", range(0, 32, 3)),
                                       ("cfg4", range(1, 64, 7)), ("cfg5", range(0, 256, 37))])
def test_workloads_with_planted_accept_lengths(binding, name, seqs):
    cfg = synth.CONFIGS[name]
    inp = synth.make_inputs(cfg, sequences=seqs)
    x, n = planted_tokens(inp.target_logits, seed=cfg.index)
    ref = run_and_compare(binding, inp.target_logits, x)
    np.testing.assert_array_equal(ref.accept_len, n)          # the plant is what the oracle finds
    # and with the tokens the sampling workloads carry (drawn from the draft distribution)
    run_and_compare(binding, inp.target_logits, inp.draft_tokens)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,k,V", [(3, 1, 1), (2, 3, 7), (5, 2, 1000), (4, 4, 4099), (2, 6, 65536 + 8),
                                   (7, 5, 32768), (1, 64, 513), (300, 2, 260)])
def test_ragged_shapes(binding, dtype, B, k, V):
    """Rows shorter than one item, rows that are not whole 16-byte vectors (element-wise path),
    rows that end inside an item, the largest k, more sequences than blocks."""
    cfg = synth.custom_config(B, k, V, dtype=dtype, recipe="gauss")
    inp = synth.make_inputs(cfg)
    x, n = planted_tokens(inp.target_logits, seed=B * 131 + k)
    ref = run_and_compare(binding, inp.target_logits, x)
    if V > 1:
        np.testing.assert_array_equal(ref.accept_len, n)


def test_ties_go_to_the_smallest_index_and_special_values(binding):
    B, k, V = 6, 3, 3 * 8192 + 12        # several items per row, ragged last item
    rng = np.random.default_rng(7)
    T = rng.standard_normal((B, k + 1, V)).astype(np.float32)
    T[0, 0, [5, 9000, 20000]] = 9.0                  # equal maxima in different items
    T[0, 1, [V - 1, V - 2]] = 9.0                    # in the ragged tail
    T[0, 2, :] = -np.inf                             # nothing above -inf: argmax 0
    T[0, 3, :] = -np.inf; T[0, 3, 12345] = -1e30     # one finite entry
    T[1, 0, 100] = np.inf; T[1, 0, 50] = np.inf      # +inf twice
    T[1, 1, :] = 0.0; T[1, 1, 17] = -0.0             # zeros of both signs are equal
    T[1, 2, :] = -3.0                                # a constant row
    T[2, 0, 7] = np.nan; T[2, 0, 8] = 50.0           # NaN is ignored
    T[2, 1, :] = np.nan                              # nothing comparable: argmax 0
    T[3, :, :] = -np.abs(T[3, :, :]) - 1.0           # all negative
    T[3, 1, 4] = -1e-45                              # a negative subnormal as the maximum
    x = rng.integers(0, V, size=(B, k)).astype(np.int32)
    x[0] = [5, V - 2, 0]
    x[1] = [50, 0, 0]
    x[2] = [8, 0, 3]
    ref = run_and_compare(binding, T, x)
    assert list(ref.argmax[0]) == [5, V - 2, 0, 12345]
    assert list(ref.argmax[1][:3]) == [50, 0, 0]
    assert ref.accept_len[0] == 3 and ref.accept_len[1] == 3 and ref.accept_len[2] == 2
    # the same through bf16 (values above are exactly representable or stay ordered)
    Tb = synth.f32_to_bf16_bits(np.nan_to_num(T, nan=-7.0))
    run_and_compare(binding, Tb, x)


def test_tokens_outside_the_vocabulary_match_nothing(binding):
    cfg = synth.custom_config(4, 3, 2048, dtype="f32")
    inp = synth.make_inputs(cfg)
    x = np.array([[-1, 0, 0], [2048, 0, 0], [2 ** 31 - 1, 0, 0], [-2 ** 31, 0, 0]], np.int32)
    ref = run_and_compare(binding, inp.target_logits, x)
    assert (ref.accept_len == 0).all()


def test_caller_workspace_no_argmax_and_back_to_back_calls(binding):
    cfg = synth.custom_config(9, 4, 50000, dtype="bf16", recipe="peaks")
    inp = synth.make_inputs(cfg)
    x, _ = planted_tokens(inp.target_logits, seed=3)
    need = binding.sd_greedy_workspace_bytes(cfg.B, cfg.k)
    assert need > 0
    ws = torch.full((need,), 0xAB, dtype=torch.uint8, device="cuda")      # dirty on purpose
    for _ in range(3):
        run_and_compare(binding, inp.target_logits, x, workspace=ws, want_argmax=False)
    with pytest.raises(binding.SdVerifyError):
        binding.sd_verify_greedy(device_logits(inp.target_logits), torch.from_numpy(x).cuda(),
                                 workspace=ws[: need - 256])


def test_interleaves_with_the_sampling_entry_point_on_the_library_scratch(binding):
    """Both entry points use the library's scratch when given none; neither may disturb the other."""
    cfg = synth.CONFIGS["cfg2"]
    inp = synth.make_inputs(cfg)
    T = device_logits(inp.target_logits)
    D = device_logits(inp.draft_logits)
    xs = torch.from_numpy(inp.draft_tokens).cuda()
    u = torch.from_numpy(inp.uniforms).cuda()
    first = binding.sd_verify_feedback(T, D, xs, u, inp.tau)
    torch.cuda.synchronize()
    big = synth.custom_config(64, 7, 4096, dtype="f32")
    inp2 = synth.make_inputs(big)
    x2, _ = planted_tokens(inp2.target_logits, seed=11)
    for _ in range(2):
        run_and_compare(binding, inp2.target_logits, x2)
        again = binding.sd_verify_feedback(T, D, xs, u, inp.tau)
        torch.cuda.synchronize()
        assert torch.equal(again.accept_len, first.accept_len)
        assert torch.equal(again.tokens, first.tokens)
        assert torch.equal(again.loss, first.loss)


def test_full_size_cfg5_sampled_rows(binding):
    """The bench shape (B=256, k=6, V=128256, fp32): all outputs against the oracle, which finishes
    this one in seconds since it reads every logit once."""
    cfg = synth.CONFIGS["cfg5"]
    inp = synth.make_inputs(cfg)
    x, n = planted_tokens(inp.target_logits, seed=5)
    ref = run_and_compare(binding, inp.target_logits, x)
    np.testing.assert_array_equal(ref.accept_len, n)
