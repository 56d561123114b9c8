"""How well the distillation objective predicts a drafter's acceptance.

    python -m paper_2512_15773_b200.drafter_quality [--workload pusht_xfmr] [--chunks 256] [--K 8]

The drafter is trained (outside this library) by minimising L = lambda1 L_pred + lambda2 L_norm against the frozen
base model (Sec. 3.2).  L_norm is the mean squared offset of the drafter's posterior mean in units of sigma_t, and a
draft whose mean is off by d is accepted by the test of Sec. 3.1 with probability 2 Phi(-|d| / 2); so the objective
itself predicts the acceptance rate a drafter will see.  For drafter / base pairs of growing mismatch (seeded random
networks whose output heads are scaled by gamma) this script evaluates the objective on clean chunks drawn from the
base model (tsdp_distill_loss), then runs the speculative sampler and prints the acceptance it measured beside the
prediction.  One JSON line per gamma.
"""
import argparse
import json

import numpy as np


def main():
    import torch
    from . import binding, inputs
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="pusht_xfmr")
    ap.add_argument("--chunks", type=int, default=256)
    ap.add_argument("--K", type=int, default=8)
    ap.add_argument("--gammas", default="0.01,0.02,0.05,0.1,0.2,0.5,1.0")
    args = ap.parse_args()
    N, K = args.chunks, args.K
    acc = binding.AcceptT(0, 1.0, 1.0, 1)
    for gamma in [float(g) for g in args.gammas.split(",")]:
        wl = dict(inputs.WORKLOADS[args.workload], gamma=gamma)
        cfg = binding.make_config(wl["H"], wl["A"], wl["To"], wl["Do"], wl["base"], wl["draft"], T=wl["T"], max_B=N,
                                  max_K=max(K, 1), precision=wl["precision"])
        smp = binding.Sampler(cfg)
        smp.load_weights(binding.BASE, inputs.make_net(1, wl, "base"))
        smp.load_weights(binding.DRAFT, inputs.make_net(2, wl, "draft"))
        obs = torch.tensor(inputs.make_obs(3, N, wl["To"], wl["Do"]).astype(np.float32), device="cuda")
        x0 = torch.zeros(N, wl["H"], wl["A"], device="cuda")
        smp.sample_chunk(obs, N, 0, acc, 11, x0)                      # clean chunks: vanilla samples of the base model
        L_pred, L_norm, L, p_acc = smp.distill_loss(x0, obs, N, 12)
        out = torch.zeros_like(x0)
        smp.reset_stats()
        smp.sample_chunk(obs, N, K, acc, 13, out)
        st = smp.stats()
        print(json.dumps(dict(workload=args.workload, gamma=gamma, L_pred=L_pred, L_norm=L_norm,
                              predicted_acceptance=p_acc, measured_acceptance=st["drafts_accepted"] / max(st["drafts_tested"], 1),
                              accepted_per_drafted=st["drafts_accepted"] / max(st["draft_evals"], 1),
                              base_forwards_per_chunk=st["env_rounds"] / N)))
        smp.close()


if __name__ == "__main__":
    main()
