"""Halo pack/unpack microbenchmark (2D blocks of 64^2 .. 4096^2, halo width 1 and 4; one 3D case).

    python -m paper_2210_01238_b200.halo_bench [--total-gib 1.0] [--sizes 64 256 1024 4096] [--no-3d]

For a block edge B the domain is a G x G grid of blocks (G = 64, 32, 8, 4) so that every kind of
face has interior instances: 4 G (G-1) faces are exchanged per call.  Data: Uniform[-1,1], seed 2.
The 3D case is the 1024^3 domain in 128^3 blocks (2688 faces, 352 MB of face payload per exchange).
Each operation (pack, unpack, pack then unpack; per face direction and for all faces; for all
faces also the exchange that does pack and unpack in one launch) is repeated until `--total-gib`
of face payload has moved, and reported as

    GB/s = counted bytes x repetitions / time,

counted bytes = 16 per face cell for a pack or an unpack (8 read + 8 written), 32 for pack then
unpack, 24 for the one-launch exchange (one read, two writes), and as that rate over the measured
copy bandwidth of the device (`roofline`; faces that are strided columns move a 32-byte sector per
8 useful bytes, so the x faces cannot come near it).

"hot": repetitions back to back (the faces stay in L2 when the payload is far below 126 MB);
"cold": an L2-evicting write between repetitions, only the operation itself timed with CUDA
events -- in a real sweep the faces were streamed out of the cache long before the pack.
Prints one JSON line per case and a table on stderr.
"""
from __future__ import annotations

import argparse
import json
import math
import sys

from . import inputs, jac

COUNTED_BYTES_PER_CELL = {"pack": 16, "unpack": 16, "pack+unpack": 32, "exchange": 24}


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


def _case(torch, stream, flush, n, b, h, total_gib, peak_gbs, dense):
    """All operations on one decomposition; returns the record."""
    ndim = len(n)
    g = [nn // bb for nn, bb in zip(n, b)]
    cells = {}
    for axis, name in enumerate("xyz"[:ndim]):
        faces = 2 * (g[axis] - 1) * math.prod(g[a] for a in range(ndim) if a != axis)
        cells[name] = faces * h * math.prod(b[a] for a in range(ndim) if a != axis)
    cells["all"] = sum(cells.values())
    masks = {name: 0b11 << (2 * axis) for axis, name in enumerate("xyz"[:ndim])}
    masks["all"] = (1 << (2 * ndim)) - 1
    rec = {"grid": list(n), "block": list(b), "halo": h, "payload_bytes_per_call": 8 * cells["all"]}
    with jac.Jacobi(n, b, h, False, "exchange") as J:
        J.set_u_device(dense)
        for kind, mask in masks.items():
            reps = max(3, math.ceil(total_gib * 2 ** 30 / (8 * cells[kind])))
            ops = {"pack": lambda m=mask: J.pack_faces(m),
                   "unpack": lambda m=mask: J.unpack_faces(m),
                   "pack+unpack": lambda m=mask: (J.pack_faces(m), J.unpack_faces(m))}
            if kind == "all":
                ops["exchange"] = lambda: J.exchange_halos()
            for name, fn in ops.items():
                counted = COUNTED_BYTES_PER_CELL[name] * cells[kind]
                th = _time_hot(torch, stream, fn, reps)
                tc = _time_cold(torch, stream, fn, reps, flush)
                rec[f"{kind}:{name}"] = {
                    "reps": reps, "hot_us": th * 1e6, "cold_us": tc * 1e6, "counted_bytes": counted,
                    "hot_gbs": counted / th / 1e9, "cold_gbs": counted / tc / 1e9,
                    "roofline": {"bound": "hbm", "achieved": counted / tc / 1e9, "peak": peak_gbs, "unit": "GB/s",
                                 "frac": counted / tc / 1e9 / peak_gbs, "timing": "cold"}}
    return rec


def run(sizes, widths, total_gib, peak_gbs, with_3d=True, echo=False):
    import torch
    stream = torch.cuda.current_stream()
    flush = torch.empty(64 * 1024 * 1024, dtype=torch.float64, device="cuda")
    rows = []
    for B in sizes:
        G = inputs.HALO_BENCH_SHAPES[B]
        n = (B * G, B * G)
        dense = torch.from_numpy(inputs.uniform_field(n, inputs.HALO_BENCH_SEED)).cuda()
        for h in widths:
            rec = _case(torch, stream, flush, n, (B, B), h, total_gib, peak_gbs, dense)
            rows.append(rec)
            if echo:
                print(json.dumps(rec), flush=True)
        del dense
    if with_3d:
        n, b = (1024, 1024, 1024), (128, 128, 128)
        gen = torch.Generator(device="cuda").manual_seed(inputs.HALO_BENCH_SEED)
        dense = torch.rand((n[2], n[1], n[0]), dtype=torch.float64, device="cuda", generator=gen) * 2 - 1
        rec = _case(torch, stream, flush, n, b, 1, total_gib, peak_gbs, dense)
        rows.append(rec)
        if echo:
            print(json.dumps(rec), flush=True)
        del dense
    hdr = f"{'block':>14} {'h':>2} {'payload MB':>10} | " + " | ".join(
        f"{k:>24}" for k in ("x pack hot/cold GB/s", "y pack hot/cold GB/s", "all p+u hot/cold GB/s",
                             "one launch hot/cold us", "one launch / p+u time"))
    print(hdr, file=sys.stderr)
    for r in rows:
        pu, ex = r["all:pack+unpack"], r["all:exchange"]
        cells = [f"{r[k]['hot_gbs']:>11.0f} /{r[k]['cold_gbs']:>10.0f}" for k in ("x:pack", "y:pack", "all:pack+unpack")]
        cells.append(f"{ex['hot_us']:>11.1f} /{ex['cold_us']:>10.1f}")
        cells.append(f"{ex['hot_us'] / pu['hot_us']:>11.2f} /{ex['cold_us'] / pu['cold_us']:>10.2f}")
        print(f"{'x'.join(map(str, r['block'])):>14} {r['halo']:>2} {r['payload_bytes_per_call'] / 1e6:>10.2f} | "
              + " | ".join(cells), file=sys.stderr)
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--sizes", type=int, nargs="*", default=sorted(inputs.HALO_BENCH_SHAPES))
    ap.add_argument("--widths", type=int, nargs="*", default=list(inputs.HALO_BENCH_WIDTHS))
    ap.add_argument("--total-gib", type=float, default=1.0)
    ap.add_argument("--peak-gbs", type=float, default=6540.8,
                    help="copy bandwidth the roofline fractions are taken against (GB/s)")
    ap.add_argument("--no-3d", action="store_true")
    args = ap.parse_args()
    run(args.sizes, args.widths, args.total_gib, args.peak_gbs, not args.no_3d, echo=True)


if __name__ == "__main__":
    main()
