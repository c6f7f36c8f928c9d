"""Compress-once frameworks against CPR-P2P (Sec. III-A-1), on the GPU: error by hop count and time.

    python -m paper_2304_03890_b200.compare_p2p [--P 8] [--shape 128x256x256]

Prints, for a broadcast of one smooth field over P virtual ranks and an all-reduce of P such fields, the
largest and the RMS error (in units of the bound) of the ranks grouped by how many compress/decompress pairs
their copy went through, and the device time of each replay.  Everything runs through the C ABI.
"""
import argparse

import torch

from . import binding as B
from . import fields


def timed(fn, reps=5):
    fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def err_by_group(out, exact, eb, group_of):
    rows = {}
    for r in range(out.shape[0]):
        d = (out[r].double() - exact).abs()
        g = group_of(r)
        mx, ms, k = rows.get(g, (0.0, 0.0, 0))
        rows[g] = (max(mx, float(d.max()) / eb), ms + float((d * d).mean()), k + 1)
    return {g: (mx, (ms / k) ** 0.5 / eb, k) for g, (mx, ms, k) in sorted(rows.items())}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--P", type=int, default=8)
    ap.add_argument("--shape", default="128x256x256")
    args = ap.parse_args()
    P = args.P
    shape = tuple(int(v) for v in args.shape.split("x"))

    # broadcast
    cfg = fields.config2(device="cuda", shape=shape, sigma=8.0)
    x, eb = cfg["x"].reshape(-1), float(cfg["eb"])
    n = x.numel() // 4 * 4
    x = x[:n].contiguous()
    B.ensure_workspace(n, P)
    out = torch.zeros((P, n), device="cuda")
    cb = torch.zeros(P, dtype=torch.int64, device="cuda")
    t_frame = timed(lambda: B.ccoll_bcast_sim(x, out, n, P, eb, B.BCAST, cb))
    frame = out.clone()
    t_p2p = timed(lambda: B.ccoll_bcast_sim_p2p(x, out, n, P, eb))
    assert B.ccoll_get_status() == B.OK
    print(f"broadcast of {n} values to {P} ranks, eb = {eb:.4g}")
    print(f"  compress-once: {t_frame:.3f} ms, 1 compression of the buffer;  CPR-P2P: {t_p2p:.3f} ms, "
          f"{P - 1} compressions (one per receiving rank), {max(bin(r).count('1') for r in range(P))} on the longest path")
    for name, o in (("compress-once", frame), ("CPR-P2P", out)):
        depth = (lambda r: min(bin(r).count("1"), 1)) if name == "compress-once" else (lambda r: bin(r).count("1"))
        for g, (mx, rms, k) in err_by_group(o, x.double(), eb, depth).items():
            print(f"  {name:14s} {g} compressions: {k} ranks, max err {mx:.3f} eb, rms err {rms:.4f} eb")

    # all-reduce
    xs = torch.stack([fields.smooth_field(shape, 4.0, -1.0, 1.0, fields.seed_for(3, r), "cuda").reshape(-1)[:n]
                      for r in range(P)]).contiguous()
    eb = 1e-4
    exact = xs.double().sum(dim=0)
    o1, o2 = torch.empty_like(xs), torch.empty_like(xs)
    moved = torch.zeros(1, dtype=torch.int64, device="cuda")
    t_frame = timed(lambda: B.ccoll_allreduce_sim(xs, o1, eb, moved))
    t_p2p = timed(lambda: B.ccoll_allreduce_sim_p2p(xs, o2, eb, moved))
    assert B.ccoll_get_status() == B.OK
    C = B.ccoll_chunk_len(n, P)
    print(f"all-reduce (Sum) of {P} x {n} values, eb = {eb:.4g}")
    print(f"  compress-once allgather: {t_frame:.3f} ms;  CPR-P2P allgather: {t_p2p:.3f} ms")
    for name, o in (("compress-once", o1), ("CPR-P2P", o2)):
        rows = {}
        for c in range(P):
            lo, hi = min(c * C, n), min((c + 1) * C, n)
            if hi == lo:
                continue
            for r in range(P):
                h = (r - (c - 1)) % P              # hops behind the chunk's owner
                g = h if name == "CPR-P2P" else min(h, 1)
                d = (o[r, lo:hi].double() - exact[lo:hi]).abs()
                mx, ms, k = rows.get(g, (0.0, 0.0, 0))
                rows[g] = (max(mx, float(d.max()) / eb), ms + float((d * d).mean()), k + 1)
        for g, (mx, ms, k) in sorted(rows.items()):
            print(f"  {name:14s} {g} hops after the owner: max err {mx:.3f} eb, rms err {(ms / k) ** 0.5 / eb:.4f} eb")


if __name__ == "__main__":
    main()
