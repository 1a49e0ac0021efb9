"""Runs every entry point on tiny, ragged and multi-stage shapes through whichever build of the library
SD_VERIFY_LIBRARY names, compares with the CPU oracle, and prints what sd_bounds_report counted.
Started as a child process by test_bounds_checked_gpu.py (the library is chosen at import)."""
import json
import sys

import numpy as np
import torch

from oracle import sd_oracle
from paper_2603_12617_b200 import binding as b, shard, synth
from test_parity_gpu import check, oracle_of, to_device


def main():
    assert b.sd_bounds_report() is not None, "this build of the library has no range checks"
    shapes = [(2, 2, 5, "f32"), (3, 1, 17, "bf16"), (2, 3, 1023, "f32"), (4, 2, 1024, "bf16"), (5, 3, 7168 + 256, "f32"),
              (3, 2, 50000, "bf16"), (9, 3, 65536, "f32"), (2, 64, 520, "f32"), (40, 2, 16392, "bf16")]
    for (B, k, V, dt) in shapes:
        cfg = synth.custom_config(B, k, V, dtype=dt, tau=0.9, index=90)
        inp = synth.make_inputs(cfg)
        T, D, x, u = to_device(inp)
        ref = oracle_of(inp)
        for cluster in (0, 3, 8):
            b.sd_set_option(b.SD_OPT_CLUSTER, cluster)
            check(inp, b.sd_verify_feedback_ex(T, D, x, u, inp.tau), ref, max_band_frac=1.0)
        b.sd_set_option(b.SD_OPT_CLUSTER, 0)
        check(inp, b.sd_verify_feedback(T, D, x, u, inp.tau), ref, max_band_frac=1.0)
        h = b.sd_verify_feedback_hint(T, D, x, u, inp.tau, torch.zeros_like(D))
        check(inp, h, ref, max_band_frac=1.0)
        es = T.element_size()
        if (V * es) % 16 == 0:
            e = b.sd_verify_error_feedback(T, D, x, u, inp.tau)
            assert torch.equal(e.accept_len, h.accept_len)
        g = b.sd_verify_greedy(T, x)
        gref = sd_oracle.verify_greedy(inp.target_logits, inp.draft_tokens)
        assert (g.accept_len.cpu().numpy() == gref.accept_len).all() and (g.tokens.cpu().numpy() == gref.tokens).all()
        if (V * es) % 16 == 0:
            b.sd_ensemble_feedback(T, [D, D.clone()], inp.tau, 10.0)
            if V // (16 // es) >= 2:
                code = b.SD_DTYPE_F32 if dt == "f32" else b.SD_DTYPE_BF16
                cuts = shard.vocab_cuts(V, 2, es)
                Ts = [T[:, :, a:c].contiguous() for a, c in cuts]
                Ds = [D[:, :, a:c].contiguous() for a, c in cuts]
                ws = [torch.empty(max(256, b.sd_vp_workspace_bytes(B, k, c - a, code)), dtype=torch.uint8, device="cuda")
                      for a, c in cuts]
                recs = torch.stack([b.sd_vp_partial(Ts[r], Ds[r], x, inp.tau, cuts[r][0], V, ws[r]) for r in range(2)], 0).contiguous()
                fins = [b.sd_vp_finish(Ts[r], Ds[r], x, u, inp.tau, cuts[r][0], V, recs, 2, r, ws[r]) for r in range(2)]
                m = torch.stack([f.local_mass for f in fins], 0).contiguous()
                for r in range(2):
                    b.sd_vp_draw(Ts[r], Ds[r], x, u, inp.tau, cuts[r][0], V, fins[r].accept_len, m, 2, r, fins[r].status, ws[r])
        torch.cuda.synchronize()
    print("REPORT " + json.dumps(b.sd_bounds_report()))


if __name__ == "__main__":
    sys.exit(main())
