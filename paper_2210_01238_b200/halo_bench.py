"""Halo pack/unpack microbenchmark (2D blocks of 64^2 .. 4096^2, halo width 1 and 4).

    python -m paper_2210_01238_b200.halo_bench [--total-gib 1.0] [--sizes 64 256 1024 4096]

For a block edge B the domain is a G x G grid of blocks (G = 64, 32, 8, 4) so that every kind of
face has interior instances: 4 G (G-1) faces are exchanged per call.  Data: Uniform[-1,1], seed 2.
Each operation (pack, unpack, pack+unpack; x faces = strided columns, y faces = contiguous rows,
all faces; for all faces also the exchange that does pack and unpack in one launch, counted with
the bytes of pack + unpack) is repeated until `--total-gib` of face payload has moved, and reported as

    GB/s = 2 x payload x repetitions / time          (read + write of every face cell)

"hot": repetitions back to back (the faces stay in L2: payloads are far below 126 MB);
"cold": an L2-evicting write between repetitions, only the operation itself timed with CUDA
events -- in a real sweep the faces were streamed out of the cache long before the pack.
Prints one JSON line per (block, halo) and a table on stderr.
"""
from __future__ import annotations

import argparse
import json
import math
import sys

import numpy as np

from . import inputs, jac

X_FACES, Y_FACES, ALL_FACES = 0b0011, 0b1100, 0b1111


def _time_hot(torch, stream, fn, reps):
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fn()
    torch.cuda.synchronize()
    a.record(stream)
    for _ in range(reps):
        fn()
    b.record(stream)
    torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e-3 / reps


def _time_cold(torch, stream, fn, reps, flush):
    total = 0.0
    reps = min(reps, 40)
    for _ in range(reps):
        flush.fill_(1.0)                       # 512 MB write: evicts the 126 MB L2
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        torch.cuda.synchronize()
        total += a.elapsed_time(b) * 1e-3
    return total / reps


def run(sizes, widths, total_gib):
    import torch
    stream = torch.cuda.current_stream()
    flush = torch.empty(64 * 1024 * 1024, dtype=torch.float64, device="cuda")
    rows = []
    for B in sizes:
        G = inputs.HALO_BENCH_SHAPES[B]
        n = (B * G, B * G)
        dense = torch.from_numpy(inputs.uniform_field(n, inputs.HALO_BENCH_SEED)).cuda()
        for h in widths:
            with jac.Jacobi(n, (B, B), h, False, "exchange") as J:
                J.set_u_device(dense)
                faces_per_kind = 2 * G * (G - 1)
                payload = {"x": faces_per_kind * B * h * 8, "y": faces_per_kind * B * h * 8}
                payload["all"] = payload["x"] + payload["y"]
                rec = {"block": B, "grid": G, "halo": h, "payload_bytes_per_call": payload["all"]}
                for kind, mask in (("x", X_FACES), ("y", Y_FACES), ("all", ALL_FACES)):
                    reps = max(3, math.ceil(total_gib * 2 ** 30 / payload[kind]))
                    ops = {"pack": lambda m=mask: J.pack_faces(m),
                           "unpack": lambda m=mask: J.unpack_faces(m),
                           "pack+unpack": lambda m=mask: (J.pack_faces(m), J.unpack_faces(m))}
                    if kind == "all":     # the same end state from one launch; counted like pack + unpack
                        ops["exchange"] = lambda: J.exchange_halos()
                    for name, fn in ops.items():
                        mult = 2 if name in ("pack+unpack", "exchange") else 1
                        th = _time_hot(torch, stream, fn, reps)
                        tc = _time_cold(torch, stream, fn, reps, flush)
                        rec[f"{kind}:{name}"] = {
                            "reps": reps, "hot_us": th * 1e6, "cold_us": tc * 1e6,
                            "hot_gbs": 2 * mult * payload[kind] / th / 1e9,
                            "cold_gbs": 2 * mult * payload[kind] / tc / 1e9}
                rows.append(rec)
                print(json.dumps(rec), flush=True)
    hdr = f"{'block':>6} {'h':>2} {'faces':>6} {'payload MB':>10} | " + " | ".join(
        f"{k:>22}" for k in ("x pack hot/cold GB/s", "y pack hot/cold GB/s", "all p+u hot/cold GB/s",
                             "one launch hot/cold"))
    print(hdr, file=sys.stderr)
    for r in rows:
        cells = [r["x:pack"], r["y:pack"], r["all:pack+unpack"], r["all:exchange"]]
        print(f"{r['block']:>6} {r['halo']:>2} {4 * r['grid'] * (r['grid'] - 1):>6} "
              f"{r['payload_bytes_per_call'] / 1e6:>10.2f} | " +
              " | ".join(f"{c['hot_gbs']:>10.0f} /{c['cold_gbs']:>9.0f}" for c in cells), file=sys.stderr)
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--sizes", type=int, nargs="*", default=sorted(inputs.HALO_BENCH_SHAPES))
    ap.add_argument("--widths", type=int, nargs="*", default=list(inputs.HALO_BENCH_WIDTHS))
    ap.add_argument("--total-gib", type=float, default=1.0)
    args = ap.parse_args()
    run(args.sizes, args.widths, args.total_gib)


if __name__ == "__main__":
    main()
