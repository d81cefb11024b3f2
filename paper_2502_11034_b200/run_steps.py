"""Run a few fused AdaGC + AdamW steps (or clip-only steps) on a named synthetic layout.

    python -m paper_2502_11034_b200.run_steps --workload gpt2_small --steps 4 [--mode step|clip|lion|sgdm] [--n-layer N]
        [--update-path auto|registers|bulk] [--fused-small] [--state f32|bf16] [--separate-finalize]

A minimal driver of the C ABI (adagc_create / adagc_step / adagc_clip / adagc_get_stats): useful as
an example and as a small, short-running target for profilers.  Prints the per-phase device times.
"""
from __future__ import annotations

import argparse

import torch

from . import binding, workloads


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="gpt2_small")
    ap.add_argument("--steps", type=int, default=4)
    ap.add_argument("--mode", choices=["step", "clip", "lion", "sgdm"], default="step")
    ap.add_argument("--n-layer", type=int, default=None, help="override the layer count of a layered layout")
    ap.add_argument("--warmup", type=int, default=1, help="T_start: steps of global-norm clipping")
    ap.add_argument("--update-path", choices=["auto", "registers", "bulk"], default="auto",
                    help="kernel of the update phase (adagc_desc.flags)")
    ap.add_argument("--fused-small", action="store_true",
                    help="ADAGC_FUSED_SMALL: adagc_step as one cooperative kernel (small layouts, --mode step)")
    ap.add_argument("--state", choices=["f32", "bf16"], default="f32", help="dtype of the m and v arenas (adagc_desc.state_dtype)")
    ap.add_argument("--separate-finalize", action="store_true",
                    help="ADAGC_SEPARATE_FINALIZE: the per-tensor decisions of AdaGC steps in a kernel of their own")
    args = ap.parse_args()
    over = {} if args.n_layer is None else {"n_layer": args.n_layer}
    wl = workloads.build(args.workload, **over)
    hp = wl.hyper
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    flags = {"auto": binding.UPDATE_PATH_AUTO, "registers": binding.UPDATE_PATH_REGISTERS,
             "bulk": binding.UPDATE_PATH_BULK}[args.update_path]
    if args.fused_small:
        flags |= binding.FUSED_SMALL
    if args.separate_finalize:
        flags |= binding.SEPARATE_FINALIZE
    sd = torch.bfloat16 if args.state == "bf16" else torch.float32
    opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], device=dev, flags=flags, state_dtype=sd)
    theta = workloads.init_params(wl, dev)
    m = torch.zeros(wl.arena_elems, dtype=sd, device=dev)
    v = torch.zeros_like(m)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device=dev)
    g = workloads.grads_for_step(wl, 1, dev)
    g_out = torch.empty_like(g) if args.mode == "clip" else None
    opt.set_phase_timing(True)
    for t in range(1, args.steps + 1):
        if args.mode == "step":
            opt.step(theta, g, m, v, ema, t, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"],
                     hp["lambda_rel"], hp["beta"], args.warmup)
        elif args.mode == "lion":
            opt.step_lion(theta, g, m, ema, t, 1e-4, 0.9, 0.99, hp["wd"], hp["lambda_rel"], hp["beta"], args.warmup)
        elif args.mode == "sgdm":
            opt.step_sgdm(theta, g, m, ema, t, 1e-2, 0.9, hp["wd"], hp["lambda_rel"], hp["beta"], args.warmup)
        else:
            opt.clip(g, g_out, ema, t, hp["lambda_rel"], hp["beta"], args.warmup)
        ms = opt.get_phase_times()
        print(f"step {t}: norm {ms[0]:.4f} ms, finalize {ms[1]:.4f} ms, {'scale' if args.mode == 'clip' else 'update'} "
              f"{ms[2]:.4f} ms  ({wl.n_params} params)")
    st = opt.get_stats()
    print(f"steps_done={st['steps_done']} clipped_last_step={int(st['flag'].sum())} status={st['status']} "
          f"kernels_launched={opt.launch_count()}")
    opt.close()


if __name__ == "__main__":
    main()
