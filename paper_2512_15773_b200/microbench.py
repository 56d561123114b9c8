"""Kernel-level timing of the tensor-core GEMM on the shapes a workload's verification forward uses.

    python -m paper_2512_15773_b200.microbench [--workload serving_xfmr] [--batch 256] [--K 10] [--reps 20]

Every linear layer of one transformer block of the base model is timed on M = batch * (K+1) * H token
rows: `reps` launches back to back between one pair of CUDA events (tsdp_gemm_timed).  Operands of
consecutive launches are the same, so whatever fits the L2 stays there, as it does inside the forward
pass where each operand was written by the previous kernel.  Prints one line per shape and one JSON
line with the flop-weighted total of the six plain shapes, and the total of the four kernels the decoder
transformer really launches per block (QKV projection with the self-attention in its epilogue, the bf16
attention projection, MLP up, MLP down: the cross-attention projections are folded into its memory tokens).
With --library each plain shape is also timed as torch.mm (the vendor library's bf16 GEMM, no bias, no epilogue) on
the same operands: context for what the shape itself allows, not a path of the sampler.
"""
import argparse
import json

import numpy as np


def block_shapes(d):
    """(name, N, K, epilogue) of the GEMMs of one pre-LN block, in launch order."""
    return [("qkv", 3 * d, d, 0), ("qkv_attn", 3 * d, d, 4), ("attn_out", d, d, 2), ("attn_out_bf16", d, d, 0), ("q_cross", d, d, 0),
            ("cross_out", d, d, 2), ("mlp_up", 4 * d, d, 1), ("mlp_down", d, 4 * d, 2)]


def main():
    import torch
    from . import binding, inputs
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="serving_xfmr")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--K", type=int, default=-1)
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--library", action="store_true", help="also time torch.mm on the same operands")
    args = ap.parse_args()
    wl = dict(inputs.WORKLOADS[args.workload])
    B = args.batch or wl["B"]
    K = wl["K"] if args.K < 0 else args.K
    d = wl["base"]["d"]
    M = B * (K + 1) * wl["H"]
    tiny = dict(arch="xfmr", layers=1, d=128, heads=4)
    cfg = binding.make_config(wl["H"], wl["A"], 2, 4, tiny, tiny, max_B=1, max_K=1, precision=1)   # only the GEMM is used
    smp = binding.Sampler(cfg)
    g = torch.Generator(device="cuda").manual_seed(0)
    tot_ms, tot_flop, rows = 0.0, 0.0, []
    for name, N, Kd, epi in block_shapes(d):
        A = torch.randn(M, Kd, device="cuda", generator=g).to(torch.bfloat16)
        W = (torch.randn(N, Kd, device="cuda", generator=g) / np.sqrt(Kd)).to(torch.bfloat16)
        bias = torch.randn(N, device="cuda", generator=g)
        out = torch.zeros(M, Kd if epi == 4 else N, device="cuda", dtype=torch.bfloat16 if epi in (0, 1, 4) else torch.float32)
        ms = smp.gemm_timed(A, W, bias, M, N, Kd, epi, out, args.reps)
        flop = 2.0 * M * N * Kd
        io = M * Kd * 2 + N * Kd * 2 + (M * Kd * 2 if epi == 4 else M * N * (2 if epi in (0, 1) else (8 if epi == 2 else 4)))
        rows.append(dict(name=name, M=M, N=N, K=Kd, epi=epi, us=1e3 * ms, tflops=flop / ms / 1e9, gbs=io / ms / 1e6))
        if args.library and epi != 4:
            Wt = W.t()
            lib_out = torch.empty(M, N, device="cuda", dtype=torch.bfloat16)
            for _ in range(3):
                torch.mm(A, Wt, out=lib_out)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(args.reps):
                torch.mm(A, Wt, out=lib_out)
            e1.record()
            torch.cuda.synchronize()
            lib_ms = e0.elapsed_time(e1) / args.reps
            rows[-1].update(library_us=1e3 * lib_ms, library_tflops=flop / lib_ms / 1e9)
        tot_ms += ms; tot_flop += flop
        print(f"{name:10s} M={M:6d} N={N:5d} K={Kd:5d} epi={epi}  {1e3 * ms:8.1f} us  {flop / ms / 1e9:7.1f} TFLOP/s"
              f"  {io / ms / 1e6:7.0f} GB/s (A + W + out bytes)"
              + (f"   torch.mm {rows[-1]['library_us']:8.1f} us {rows[-1]['library_tflops']:7.1f} TFLOP/s" if "library_us" in rows[-1] else ""))
    # what the decoder transformer launches per block: fused QKV + attention, the bf16 attention projection, the MLP pair
    four = [r for r in rows if r["name"] in ("qkv_attn", "attn_out_bf16", "mlp_up", "mlp_down")]
    rows_all, rows = rows, [r for r in rows if r["name"] not in ("qkv_attn", "attn_out_bf16")]
    tot_ms = sum(r["us"] for r in rows) / 1e3; tot_flop = sum(2.0 * r["M"] * r["N"] * r["K"] for r in rows)
    us4 = sum(r["us"] for r in four)
    print(json.dumps(dict(workload=args.workload, batch=B, K=K, rows=M, block_us=1e3 * tot_ms,
                          block_tflops=tot_flop / tot_ms / 1e9, folded_block_us=us4,
                          folded_block_tflops=sum(2.0 * r["M"] * r["N"] * r["K"] for r in four) / us4 / 1e6, shapes=rows_all)))
    smp.close()


if __name__ == "__main__":
    main()
