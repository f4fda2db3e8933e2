"""Run the library on seeded synthetic inputs from the command line (timing / profiling aid).

    python -m paper_2410_20926_b200.cli --op forward --dims 32,32,32 --B 1 --H 32 --H-kv 8 --D 128
    python -m paper_2410_20926_b200.cli --op backward --dims 32,32,32 --H 16 --H-kv 4 --reps 2
    python -m paper_2410_20926_b200.cli --op forward --dims 4096 --rope-base 10000 --no-fusion

q, k, v (and dout) ~ N(0,1) in bf16, drawn on the device with a fixed seed.  Prints one JSON line:
the launch plan, the CUDA-event time per repetition and the kernels launched.  Everything is
computed by the CUDA library through its C ABI; there is no fallback.
"""
from __future__ import annotations

import argparse
import json
import math

from . import api as ta


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--op", choices=["forward", "backward"], default="forward")
    ap.add_argument("--dims", default="32,32,32", help="tensor shape n_1,...,n_m (prod = tokens per head)")
    ap.add_argument("--B", type=int, default=1)
    ap.add_argument("--H", type=int, default=32)
    ap.add_argument("--H-kv", type=int, default=8)
    ap.add_argument("--D", type=int, default=128)
    ap.add_argument("--non-causal", action="store_true")
    ap.add_argument("--rope-base", type=float, default=0.0)
    ap.add_argument("--no-fusion", action="store_true")
    ap.add_argument("--no-tensor-core", action="store_true")
    ap.add_argument("--no-overlap", action="store_true", help="launch every hop fully serialised")
    ap.add_argument("--f32-grads", action="store_true")
    ap.add_argument("--saved-hops", action="store_true",
                    help="backward: take the hop inputs from a forward run with TA_FLAG_SAVE_HOPS instead of "
                         "recomputing them (the forward is not part of the timed repetitions)")
    ap.add_argument("--warmup", type=int, default=1)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--seed", type=int, default=1)
    args = ap.parse_args(argv)

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device (there is no CPU fallback)")
    ta.load()
    dims = [int(x) for x in args.dims.split(",")]
    N = math.prod(dims)
    B, H, Hkv, D = args.B, args.H, args.H_kv, args.D
    causal = not args.non_causal
    gen = torch.Generator(device="cuda").manual_seed(args.seed)

    def draw(heads):
        return torch.randn(B, heads, N, D, device="cuda", generator=gen).bfloat16()

    q, k, v = draw(H), draw(Hkv), draw(Hkv)
    flags = (ta.TA_FLAG_NO_HOP_FUSION if args.no_fusion else 0) | (ta.TA_FLAG_NO_TENSOR_CORE if args.no_tensor_core else 0) \
        | (ta.TA_FLAG_NO_HOP_OVERLAP if args.no_overlap else 0)
    if args.op == "forward":
        out = torch.empty_like(q)

        def step():
            ta.ta_forward_ex(q, k, v, out, B, H, Hkv, N, D, dims, causal, flags=flags, rope_base=args.rope_base)
    else:
        dout = draw(H)
        gdt = torch.float32 if args.f32_grads else torch.bfloat16
        dq = torch.empty(B, H, N, D, dtype=gdt, device="cuda")
        dk = torch.empty(B, Hkv, N, D, dtype=gdt, device="cuda")
        dv = torch.empty(B, Hkv, N, D, dtype=gdt, device="cuda")
        mode = ta.TA_WS_BACKWARD_F32_GRADS if args.f32_grads else ta.TA_WS_BACKWARD
        nbytes = ta.ta_workspace_bytes(B, H, Hkv, N, D, dims, ta.TA_DTYPE_BF16, mode)
        ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
        saved = None
        if args.saved_hops:
            nsave = ta.ta_workspace_bytes(B, H, Hkv, N, D, dims, ta.TA_DTYPE_BF16, ta.TA_WS_FORWARD_SAVE)
            saved = torch.empty(max(nsave, 256), dtype=torch.uint8, device="cuda")
            ta.ta_forward_ex(q, k, v, torch.empty_like(q), B, H, Hkv, N, D, dims, causal,
                             flags=ta.TA_FLAG_SAVE_HOPS, workspace=saved, workspace_bytes=nsave,
                             rope_base=args.rope_base)

        def step():
            ta.ta_backward_ex(dout, q, k, v, dq, dk, dv, B, H, Hkv, N, D, dims, causal,
                              grad_dtype=ta.TA_DTYPE_F32 if args.f32_grads else ta.TA_DTYPE_BF16,
                              saved_hops=saved, workspace=ws, workspace_bytes=nbytes, rope_base=args.rope_base)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    n0 = ta.ta_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.reps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ta.ta_device_status()
    plan = ta.ta_plan_describe(B, H, Hkv, N, D, dims, causal, ta.TA_DTYPE_BF16, flags).strip().splitlines()
    print(json.dumps({"op": args.op, "dims": dims, "B": B, "H": H, "H_kv": Hkv, "D": D, "causal": causal,
                      "rope_base": args.rope_base, "ms_per_rep": e0.elapsed_time(e1) / max(args.reps, 1),
                      "launches_per_rep": (ta.ta_launch_count() - n0) / max(args.reps, 1),
                      "forward_plan": plan}))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
