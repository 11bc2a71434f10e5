"""A small, self-contained case of the hot path for profilers.

    python -m paper_2305_17118_b200.profile_case --config opt66b --units 2304 --steps 3 [--compress]

Builds a handle of the given workload's shape with fewer units, fills K and V
with random values directly (no prompt is streamed, so almost no launches come
before the ones of interest), declares the cache `--rows` tokens full through
sh_restore, and runs `--steps` decode steps (with `--compress`, the cache is one
short of full, so the first step is followed by a compression).  Prints the
CUDA-event time of each step.  The outputs are not meaningful attention
results; the memory traffic and instruction mix are those of the real step.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as sh
from . import workloads as wl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="opt66b", choices=wl.CONFIG_ORDER)
    ap.add_argument("--units", type=int, default=2304)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--rows", type=int, default=None, help="live rows before the first step")
    ap.add_argument("--compress", action="store_true")
    ap.add_argument("--unordered", action="store_true",
                    help="SH_OPT_COMPACTION = 1; the cache is then filled by streaming a random prompt through sh_prefill "
                         "(the selection needs real positions), a few launches before the ones of interest")
    ap.add_argument("--chunk", type=int, default=0, help="instead of decode steps, run one prompt chunk of this many tokens")
    ap.add_argument("--chunk-kernel", type=int, default=None, help="SH_OPT_PREFILL_CHUNK value: 2 warp-level MMA, 3 tcgen05")
    ap.add_argument("--split", type=int, default=None)
    ap.add_argument("--kernel", type=int, default=None, help="1 direct loads, 2 pipelined bulk copies")
    args = ap.parse_args()
    cfg = wl.CONFIGS[args.config]
    U, d = args.units, cfg.head_dim
    torch.cuda.set_device(0)
    h = sh.Handle(cfg.B, cfg.r, cfg.w, cfg.m, U, d, cfg.dtype, split=args.split, kernel=args.kernel, auto_compress=True,
                  unordered=args.unordered, prefill_chunk=args.chunk_kernel)
    rows = args.rows if args.rows is not None else (cfg.B - 1 if args.compress else cfg.B - cfg.m // 2)
    if args.chunk:
        rows = args.rows if args.rows is not None else cfg.B - args.chunk
    # K then V sit at the start of the workspace, [U][B][row_bytes] each.
    row_bytes = {"f32": 4 * d, "f16": 2 * d, "bf16": 2 * d, "int4": d // 2}[cfg.dtype]
    kv = h.slab[h._slab_off: h._slab_off + 2 * U * cfg.B * row_bytes]
    if cfg.dtype == "int4":
        kv.random_(0x11, 0xFF)
    elif cfg.dtype == "f32":
        kv.view(torch.float32).normal_()
    else:
        kv.view(torch.float16 if cfg.dtype == "f16" else torch.bfloat16).normal_()
    g = torch.Generator(device="cuda")
    g.manual_seed(1)
    if args.unordered:
        xp = torch.randn(3, rows, U, d, generator=g, device="cuda").to(cfg.torch_dtype)
        h.prefill(xp[0], xp[1], xp[2])
        del xp
    else:
        sh.lib.sh_restore(h._h, rows, 4 * cfg.B)
    x = torch.randn(3, args.steps, U, d, generator=g, device="cuda").to(cfg.torch_dtype)
    out = torch.empty(U, d, device="cuda")
    torch.cuda.synchronize()
    if args.chunk:
        c = args.chunk
        xc = torch.randn(3, c, U, d, generator=g, device="cuda").to(cfg.torch_dtype)
        oc = torch.empty(c, U, d, device="cuda")
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        h.prefill_chunk(xc[0], xc[1], xc[2], oc)
        b.record()
        torch.cuda.synchronize()
        flops = 2 * 2 * c * (rows + (c + 1) / 2) * d * U
        byts = U * (2 * rows * row_bytes + 3 * c * row_bytes + c * d * 4)
        print(f"chunk of {c} tokens over {rows} cached rows: {a.elapsed_time(b) * 1e3:.1f} us, "
              f"{flops / 1e9:.1f} GFLOP (algorithmic), {byts / 1e6:.1f} MB")
        return
    for i in range(args.steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        h.decode_step(x[0, i], x[1, i], x[2, i], out)
        b.record()
        torch.cuda.synchronize()
        n = h.n
        print(f"step {i}: {a.elapsed_time(b) * 1e3:.1f} us, live rows now {n}, "
              f"K+V bytes read {2 * U * (rows + i + 1) * row_bytes / 1e6:.1f} MB")
    assert torch.isfinite(out).all() or cfg.dtype == "int4"


if __name__ == "__main__":
    main()
