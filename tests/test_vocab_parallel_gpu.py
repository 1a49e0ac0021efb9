"""Vocabulary-parallel step (logits sharded along the vocabulary, Sec. 4.1's multi-GPU deployment)
on ONE GPU: the shards of all ranks live side by side in this GPU's memory, each rank's three local
calls run one after another, and the exchanges between the phases are concatenations.  No call waits
for another, so nothing here depends on several kernels running at the same time.

Compared with the CPU oracle on the unsharded logits at the bars of the single-GPU step, and the
replicated outputs (accept lengths, losses, status) must be bit-identical on every rank.
"""
from types import SimpleNamespace

import numpy as np
import pytest
import torch

from oracle import sd_oracle
from paper_2603_12617_b200 import shard, synth
from test_parity_gpu import check, oracle_of, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    import __graft_entry__ as entry
    entry.build()
    from paper_2603_12617_b200 import binding as b
    return b


def run_sharded(binding, inp, G, cuts=None, want_grad=True):
    """All G ranks' calls on this GPU; returns an object shaped like the single-GPU outputs."""
    T, D, x, u = to_device(inp)
    B, k, V = inp.draft_tokens.shape[0], inp.cfg.k, inp.cfg.V
    cuts = cuts or shard.vocab_cuts(V, G, T.element_size())
    code = binding.SD_DTYPE_F32 if T.dtype == torch.float32 else binding.SD_DTYPE_BF16
    Ts = [T[:, :, a:b].contiguous() for a, b in cuts]
    Ds = [D[:, :, a:b].contiguous() for a, b in cuts]
    ws = [torch.empty(max(256, binding.sd_vp_workspace_bytes(B, k, b - a, code)), dtype=torch.uint8, device="cuda")
          for a, b in cuts]
    for w in ws:
        w.fill_(0xA5)                     # the workspace may hold anything on entry
    recs = [binding.sd_vp_partial(Ts[g], Ds[g], x, inp.tau, cuts[g][0], V, ws[g]) for g in range(G)]
    all_records = torch.stack(recs, 0).contiguous()
    fins = [binding.sd_vp_finish(Ts[g], Ds[g], x, u, inp.tau, cuts[g][0], V, all_records, G, g, ws[g],
                                 want_grad=want_grad) for g in range(G)]
    for f in fins[1:]:
        assert torch.equal(f.accept_len, fins[0].accept_len)
        assert torch.equal(f.loss.view(torch.int32), fins[0].loss.view(torch.int32))
        assert torch.equal(f.status, fins[0].status)
    all_masses = torch.stack([f.local_mass for f in fins], 0).contiguous()
    toks = [binding.sd_vp_draw(Ts[g], Ds[g], x, u, inp.tau, cuts[g][0], V, fins[g].accept_len, all_masses, G, g,
                               fins[g].status, ws[g]) for g in range(G)]
    torch.cuda.synchronize()
    stacked = torch.stack(toks, 0)
    # exactly one rank claims the extra token of a sequence; the prefix and the padding agree everywhere
    n = fins[0].accept_len.long()
    extra = torch.gather(stacked, 2, n.view(1, B, 1).expand(G, B, 1)).squeeze(2)          # [G,B]
    assert ((extra >= 0).sum(0) == 1).all(), "not exactly one owner of the extra token"
    tokens = stacked.max(0).values
    status = fins[0].status.clone()
    for f in fins[1:]:
        status |= f.status                                                            # phase 3 may add bits
    grad = torch.cat([f.grad_shard for f in fins], 2).contiguous() if want_grad else None
    for g, (a, b) in enumerate(cuts):                                                 # the owner's token is in its shard
        own = extra[g] >= 0
        assert ((extra[g][own] >= a) & (extra[g][own] < b)).all()
    return SimpleNamespace(accept_len=fins[0].accept_len, tokens=tokens, loss=fins[0].loss, grad_draft=grad,
                           acc_prob=None, status=status)


@pytest.mark.parametrize("G", [1, 2, 4, 8])
@pytest.mark.parametrize("dtype,V", [("f32", 151936), ("bf16", 32000)])
def test_shards_of_equal_width(binding, dtype, V, G):
    cfg = synth.custom_config(B=12, k=4, V=V, dtype=dtype, tau=0.8, index=70)
    inp = synth.make_inputs(cfg)
    out = run_sharded(binding, inp, G)
    check(inp, out, oracle_of(inp), max_band_frac=0.2)
    assert binding.sd_launch_info()["path"] == 6


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_shards_of_unequal_width_and_a_ragged_last_region(binding, dtype):
    V = 50000
    step = 4 if dtype == "f32" else 8
    cuts = [(0, 6 * step), (6 * step, 20008), (20008, 20008 + 2 * step), (20008 + 2 * step, V)]
    cfg = synth.custom_config(B=9, k=3, V=V, dtype=dtype, tau=1.1, recipe="peaks", index=71)
    inp = synth.make_inputs(cfg)
    out = run_sharded(binding, inp, len(cuts), cuts=cuts)
    check(inp, out, oracle_of(inp), max_band_frac=0.2)


def test_workload_shapes(binding):
    """The paper's deployment (four ranks) on two of the workloads' shapes, fewer sequences."""
    for name, seqs in [("cfg3", 16), ("cfg4", 8)]:
        base = synth.CONFIGS[name]
        inp = synth.make_inputs(base, sequences=list(range(seqs)))
        out = run_sharded(binding, inp, 4)
        check(inp, out, oracle_of(inp), max_band_frac=0.2, loss_floor=0.0, grad_floor=0.0)


def test_every_accept_length_and_every_owner(binding):
    """Draft = target on a prefix of every sequence, far off behind it: accept lengths 0..k by design;
    over the batch every rank owns a draw."""
    B, k, V, G = 48, 5, 4096, 4
    cfg = synth.custom_config(B, k, V, dtype="f32", index=72)
    inp = synth.make_inputs(cfg)
    D = inp.draft_logits.copy()
    for b in range(B):
        n = b % (k + 1)
        D[b, :n] = inp.target_logits[b, :n]
        if n < k:
            D[b, n] = -inp.target_logits[b, n]
            inp.draft_tokens[b, n] = int(np.argmax(D[b, n]))
            inp.uniforms[b, n] = 0.999
    inp.draft_logits[:] = D
    out = run_sharded(binding, inp, G)
    ref = oracle_of(inp)
    check(inp, out, ref, max_band_frac=0.2)
    assert list(ref.accept_len) == [b % (k + 1) for b in range(B)]
    tok = out.tokens.cpu().numpy()
    extra = tok[np.arange(B), out.accept_len.cpu().numpy()]
    assert set((extra // (V // G)).tolist()) == set(range(G))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_zero_residual_falls_back_to_the_target_distribution(binding, dtype):
    """q = p exactly and a forced rejection: no rank has residual mass, and the token comes from p_n."""
    V, G = 4096, 4
    cfg = synth.custom_config(B=6, k=3, V=V, dtype=dtype, tau=0.9, index=66)
    inp = synth.make_inputs(cfg)
    inp.target_logits[:] = 0
    inp.draft_logits[:] = 0
    inp.draft_tokens[1, 1] = V
    inp.draft_tokens[2, 0] = -1
    inp.draft_tokens[4, 2] = V + 5
    out = run_sharded(binding, inp, G)
    ref = oracle_of(inp)
    check(inp, out, ref, max_band_frac=1.0)
    assert out.status.cpu().numpy().tolist() == [0, 5, 5, 0, 5, 0]
    tok = out.tokens.cpu().numpy()
    for b, n in [(1, 1), (2, 0), (4, 2)]:
        t = float(inp.uniforms[b, cfg.k]) * V
        if abs(t - round(t)) > 1e-3:
            assert tok[b, n] == int(t)


def test_masked_entries_and_a_shard_without_mass(binding):
    """One shard of the target is masked to -inf entirely: it contributes nothing and never owns a draw."""
    V, G = 8192, 4
    cfg = synth.custom_config(B=10, k=3, V=V, dtype="f32", index=73)
    inp = synth.make_inputs(cfg)
    inp.target_logits[:, :, 2048:4096] = -np.inf
    inp.draft_logits[:, :, 2048:4096] = -np.inf
    x = inp.draft_tokens
    x[(x >= 2048) & (x < 4096)] -= 2048
    out = run_sharded(binding, inp, G)
    check(inp, out, oracle_of(inp), max_band_frac=0.2)
    tok = out.tokens.cpu().numpy()
    extra = tok[np.arange(cfg.B), out.accept_len.cpu().numpy()]
    assert not ((extra >= 2048) & (extra < 4096)).any()


def test_bad_token_is_reported_by_every_rank(binding):
    cfg = synth.custom_config(B=3, k=3, V=2048, dtype="f32", d_sigma=0.01, index=60)
    inp = synth.make_inputs(cfg)
    inp.draft_tokens[1, 1] = cfg.V
    inp.draft_tokens[2, 0] = -3
    out = run_sharded(binding, inp, 2)
    st = out.status.cpu().numpy()
    assert st[0] == 0 and st[1] & binding.SD_STATUS_BAD_TOKEN and st[2] & binding.SD_STATUS_BAD_TOKEN
    check(inp, out, oracle_of(inp), max_band_frac=1.0)


def test_verify_only(binding):
    cfg = synth.custom_config(B=5, k=4, V=32000, dtype="bf16", index=74)
    inp = synth.make_inputs(cfg)
    out = run_sharded(binding, inp, 4, want_grad=False)
    check(inp, out, oracle_of(inp, want_grad=False), max_band_frac=0.4)


def test_refusals(binding):
    cfg = synth.custom_config(B=2, k=2, V=4096, dtype="f32", index=75)
    inp = synth.make_inputs(cfg)
    T, D, x, u = to_device(inp)
    ws = torch.empty(1 << 16, dtype=torch.uint8, device="cuda")
    odd = T[:, :, :1002].contiguous(), D[:, :, :1002].contiguous()              # not whole 16-byte vectors
    with pytest.raises(binding.SdVerifyError) as e:
        binding.sd_vp_partial(odd[0], odd[1], x, inp.tau, 0, 4096, ws)
    assert "align" in str(e.value).lower()
    half = T[:, :, :2048].contiguous(), D[:, :, :2048].contiguous()
    with pytest.raises(binding.SdVerifyError):                                  # shard reaches past the vocabulary
        binding.sd_vp_partial(half[0], half[1], x, inp.tau, 3000, 4096, ws)
    with pytest.raises(binding.SdVerifyError):                                  # workspace too small
        binding.sd_vp_partial(half[0], half[1], x, inp.tau, 0, 4096, ws[:16])
    with pytest.raises(binding.SdVerifyError):                                  # temperature
        binding.sd_vp_partial(half[0], half[1], x, 0.0, 0, 4096, ws)
    torch.cuda.synchronize()
