"""Host side of the vocabulary-parallel step on CPU: two and three gloo ranks, each holding a shard of
the vocabulary, run `shard.vocab_parallel_step` with a plain numpy stand-in for the three local
calls (the library's kernels need a GPU; what is under test here is the order of the calls, the
rank-ordered gathers, the exclusive scan of the shares in rank order that picks the owner of the
extra token, and the final maximum over the token arrays).  The result must be the oracle's on the
unsharded logits.
"""
import os
import socket
from types import SimpleNamespace

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import sd_oracle
from paper_2603_12617_b200 import shard, synth


@pytest.mark.parametrize("V,world,eb", [(32000, 8, 2), (151936, 4, 2), (128256, 4, 4), (1000, 3, 4), (64, 4, 4)])
def test_cuts_tile_the_vocabulary_on_16_byte_boundaries(V, world, eb):
    cuts = shard.vocab_cuts(V, world, eb)
    assert cuts[0][0] == 0 and cuts[-1][1] == V and len(cuts) == world
    for (a0, a1), (b0, b1) in zip(cuts, cuts[1:]):
        assert a1 == b0
    for a, b in cuts:
        assert (a * eb) % 16 == 0 and ((b - a) * eb) % 16 == 0 and b > a
    widths = [b - a for a, b in cuts]
    assert max(widths) - min(widths) <= 16 // eb


def test_cuts_refuse_what_cannot_be_cut():
    with pytest.raises(ValueError):
        shard.vocab_cuts(1001, 2, 4)        # rows are not whole vectors
    with pytest.raises(ValueError):
        shard.vocab_cuts(8, 4, 4)           # two vectors, four ranks


class NumpyPhases:
    """The three local calls written out from the definitions in fp64 (softmax with temperature,
    p(x)/q(x) test, residual max(0, p - q), inverse CDF), for a shard of columns."""

    def partial(self, T, D, x, tau, v0, V_total, ws):
        T, D = T.numpy().astype(np.float64), D.numpy().astype(np.float64)
        B, K1, Vs = T.shape
        k = K1 - 1
        rec = np.zeros((B, K1, 6))
        rec[:, :, 0] = T.max(-1) / tau
        rec[:, :, 1] = np.exp(T / tau - rec[:, :, 0:1]).sum(-1)
        rec[:, :k, 2] = D.max(-1) / tau
        rec[:, :k, 3] = np.exp(D / tau - rec[:, :k, 2:3]).sum(-1)
        xs = x.numpy() - v0
        for b in range(B):
            for i in range(k):
                if 0 <= xs[b, i] < Vs:
                    rec[b, i, 4] = T[b, i, xs[b, i]] / tau
                    rec[b, i, 5] = D[b, i, xs[b, i]] / tau
                else:
                    rec[b, i, 4] = rec[b, i, 5] = np.nan        # "this shard does not hold the token"
        return torch.from_numpy(rec.reshape(B * K1, 6))

    def finish(self, T, D, x, u, tau, v0, V_total, all_records, world, rank, ws):
        T, D = T.numpy().astype(np.float64), D.numpy().astype(np.float64)
        B, K1, Vs = T.shape
        k = K1 - 1
        rec = all_records.numpy().reshape(world, B, K1, 6)
        mT = rec[..., 0].max(0)
        lseT = mT + np.log((rec[..., 1] * np.exp(rec[..., 0] - mT)).sum(0))
        mD = rec[:, :, :k, 2].max(0)
        lseD = mD + np.log((rec[:, :, :k, 3] * np.exp(rec[:, :, :k, 2] - mD)).sum(0))
        p = np.exp(T / tau - lseT[..., None])
        q = np.exp(D / tau - lseD[..., None])
        tx = np.nanmax(rec[:, :, :k, 4], 0)           # exactly one rank holds the token
        dx = np.nanmax(rec[:, :, :k, 5], 0)
        ratio = np.exp((tx - lseT[:, :k]) - (dx - lseD))
        acc = u.numpy()[:, :k].astype(np.float64) < np.minimum(1.0, ratio)
        n = np.where(acc.all(1), k, np.argmin(acc, 1)).astype(np.int32)
        self.mass_row = np.stack([p[b, k] if n[b] == k else np.maximum(p[b, n[b]] - q[b, n[b]], 0) for b in range(B)])
        local = np.stack([self.mass_row.sum(1), np.zeros(B)], 1)
        return SimpleNamespace(accept_len=torch.from_numpy(n), loss=None, grad_shard=None,
                               local_mass=torch.from_numpy(local), status=torch.zeros(B, dtype=torch.int32))

    def draw(self, T, D, x, u, tau, v0, V_total, accept_len, all_masses, world, rank, status, ws):
        B, K1, Vs = T.shape
        k = K1 - 1
        m = all_masses.numpy()[:, :, 0]                # [world, B]
        n = accept_len.numpy()
        tok = np.full((B, K1), -1, np.int32)
        for b in range(B):
            tok[b, :n[b]] = x.numpy()[b, :n[b]]
            t = float(u[b, k]) * m[:, b].sum()
            before = m[:rank, b].sum()                 # exclusive scan in rank order
            if before <= t < before + m[rank, b] or (rank == world - 1 and t >= before + m[rank, b]):
                cdf = before + np.cumsum(self.mass_row[b])
                y = int(np.searchsorted(cdf, t, side="right"))
                tok[b, n[b]] = v0 + min(y, Vs - 1)
        return torch.from_numpy(tok)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = synth.custom_config(B=16, k=4, V=4096, dtype="f32", tau=0.8, index=76)
        inp = synth.make_inputs(cfg, workers=1)
        v0, v1 = shard.vocab_cuts(cfg.V, world, 4)[rank]
        T = torch.from_numpy(inp.target_logits[:, :, v0:v1].copy())
        D = torch.from_numpy(inp.draft_logits[:, :, v0:v1].copy())
        x, u = torch.from_numpy(inp.draft_tokens), torch.from_numpy(inp.uniforms)
        fin, tokens = shard.vocab_parallel_step(NumpyPhases(), T, D, x, u, inp.tau, v0, cfg.V, rank, world, None)
        q.put((rank, fin.accept_len.numpy().tolist(), tokens.numpy().tolist()))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_ranks_with_vocabulary_shards_reach_the_oracles_answer(world):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = [q.get(timeout=180) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = synth.custom_config(B=16, k=4, V=4096, dtype="f32", tau=0.8, index=76)
    inp = synth.make_inputs(cfg, workers=1)
    ref = sd_oracle.verify_feedback(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, inp.tau,
                                    want_grad=False, nthreads=1)
    safe = (ref.accept_band.sum(1) == 0) & (ref.cdf_margin > 1e-6)
    assert safe.sum() >= 12
    for rank, n, tok in results:
        n, tok = np.asarray(n), np.asarray(tok)
        assert (n[safe] == ref.accept_len[safe]).all()
        assert (tok[safe] == ref.tokens[safe]).all(), f"rank {rank}"
