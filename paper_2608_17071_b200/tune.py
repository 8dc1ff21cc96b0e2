"""Offline plan tuner: writes the static plan table the library compiles in.

    python -m paper_2608_17071_b200.tune [--out csrc/kx_plan_table.inc] [--margin 0.03]

For every workload shape it sweeps plan overrides (tile width, CTA pair, ring depth,
raster group, half-width tail, split count, cluster reduction), and keeps a candidate
only if (1) its output reproduces the heuristic plan's output on the same inputs within
the library's acceptance tolerance and (2) it is faster than the incumbent by at least
`margin` (a fractional keep margin, measured interleaved with the incumbent so that
clock and thermal drift hit both alike).  Shapes whose best plan is the heuristic's get
no entry.  The result has the form of the paper's artifact for this operator (Appendix A,
Algorithm 3): a static per-M table of validated settings with a heuristic fallback.

The tuner only measures and compares; every arithmetic step runs in the CUDA kernels.
Rebuild the library afterwards (`python -m paper_2608_17071_b200.build`).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import time

HERE = os.path.dirname(os.path.abspath(__file__))
FIELDS = ("path", "block_n", "cta_pair", "split_k", "raster_group", "stages", "stream_k", "narrow_tail",
          "cluster_reduce", "k_cluster")
ATOL, RTOL = 1e-2, 1.6e-2


def m_bucket(M: int):
    """M range an entry applies to: [1,4], [5,8], [9,16], (16,32], (32,64], ... (the kernels for a few
    rows change at 4 and 32; above that, powers of two)."""
    if M <= 4:
        return 1, 4
    if M <= 8:
        return 5, 8
    if M <= 16:
        return 9, 16
    hi = 1 << (M - 1).bit_length()
    return hi // 2 + 1, hi


def candidates(M: int, N: int, K: int, kx):
    T, S = kx.KX_PATH_TILE, kx.KX_PATH_SWAP
    out = []
    if M <= 4:
        for rw in (1, 2, 4):
            for warps in (2, 3, 4, 5, 6, 8, 12, 16):
                out.append(dict(path=kx.KX_PATH_GEMV, block_n=rw, split_k=warps))
    if M <= 32:
        for rw in (16, 32):
            out.append(dict(path=kx.KX_PATH_SKINNY, block_n=rw))
    if M <= 256:
        bn = 16 if M <= 16 else 32 if M <= 32 else 64 if M <= 64 else 128 if M <= 128 else 256
        for sk in (1, 2, 3, 4, 5, 6, 8):
            out.append(dict(path=S, block_n=bn, split_k=sk))
        one_kb_swap = {16: 12, 32: 11, 64: 9, 128: 7, 256: 4}
        out.append(dict(path=S, block_n=bn, stages=one_kb_swap[bn]))
        for sk in (2, 4, 8, 12, 16):
            out.append(dict(path=S, block_n=bn, split_k=sk, cluster_reduce=1))
        if bn <= 128:
            for sk in (2, 3, 4, 6, 8):
                out.append(dict(path=S, block_n=bn, split_k=sk, cluster_reduce=3))
    if M > 64:
        for bn in (256, 192, 128, 64):
            for pair in (1, 2):
                out.append(dict(path=T, block_n=bn, cta_pair=pair))
        for rg in (2, 4, 16, 32):
            out.append(dict(path=T, block_n=256, cta_pair=2, raster_group=rg))
        out.append(dict(path=T, block_n=256, cta_pair=2, stages=5))
        out.append(dict(path=T, block_n=256, cta_pair=2, narrow_tail=1))
        # the two tails for left-over tiles, each forced (the heuristic switches at 64 k-blocks)
        for bn in (256, 192):
            out.append(dict(path=T, block_n=bn, cta_pair=2, narrow_tail=3))
            out.append(dict(path=T, block_n=bn, cta_pair=2, narrow_tail=2))
        out.append(dict(path=T, block_n=256, cta_pair=1, narrow_tail=1))
        for bn in (256, 192, 128):
            for kc in (2, 4):
                out.append(dict(path=T, block_n=bn, cta_pair=1, k_cluster=kc))
        # the variants whose ring stages hold two k-blocks (selected by their stage count)
        two_kb = {(256, 2): 3, (256, 1): 2, (192, 1): 2, (128, 1): 3, (64, 1): 4, (192, 2): 3, (128, 2): 4}
        one_kb = {(256, 2): 6, (256, 1): 4, (192, 1): 4, (128, 1): 6, (64, 1): 8, (192, 2): 6, (128, 2): 7}
        for (bn, pair), st in two_kb.items():
            out.append(dict(path=T, block_n=bn, cta_pair=pair, stages=st))
            out.append(dict(path=T, block_n=bn, cta_pair=pair, stages=one_kb[(bn, pair)]))
        for bn in (256, 128):
            out.append(dict(path=T, block_n=bn, cta_pair=1, k_cluster=2, stages=two_kb[(bn, 1)]))
            out.append(dict(path=T, block_n=bn, cta_pair=1, k_cluster=2, stages=one_kb[(bn, 1)]))
        # CTA-pair tiles whose K range is split over two pairs (a cluster of four)
        for bn in (256, 192, 128):
            out.append(dict(path=T, block_n=bn, cta_pair=2, k_cluster=2))
            out.append(dict(path=T, block_n=bn, cta_pair=2, k_cluster=2, stages=two_kb[(bn, 2)]))
        # stream-K over the last wave(s)
        for bn, pair in ((256, 2), (192, 2), (256, 1)):
            out.append(dict(path=T, block_n=bn, cta_pair=pair, stream_k=2))
    return out


def tune(margin: float, rounds: int, block_s: float, verbose: bool = True):
    import torch
    from . import binding as kx
    from . import inputs

    kx.kx_init(torch.cuda.current_device())
    dev = torch.device("cuda")
    entries, report = [], []
    for name, wl in inputs.all_workloads().items():
        M, N, K = wl.M, wl.N, wl.K
        per = wl.algorithmic_bytes
        nsets = int(max(2, min(16, (2 * 126 * (1 << 20)) // per + 1)))
        g = torch.Generator(device=dev)
        g.manual_seed(wl.seed)
        sets = []
        for _ in range(nsets):
            X = (torch.randn(M, K, device=dev, generator=g) / K ** 0.5).bfloat16()
            W = (torch.randn(N, K, device=dev, generator=g) / K ** 0.5).bfloat16()
            b = (torch.randn(N, device=dev, generator=g) * 0.1).bfloat16() if wl.has_bias else None
            R = torch.randn(M, N, device=dev, generator=g).bfloat16() if wl.has_residual else None
            sets.append((X, W, b, R, torch.empty(M, N, dtype=torch.bfloat16, device=dev)))

        def run(ov, s):
            kx.kx_outproj_residual_ex(s[0], s[1], s[2], s[3], s[4], ov)

        def block(ov, steps):
            # pre-marshalled calls: the checked Python path costs more than a small kernel runs
            calls = [kx.bound_call(s[0], s[1], s[2], s[3], s[4], ov=ov) for s in sets]
            for i in range(3):
                calls[i % nsets]()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(steps):
                calls[i % nsets]()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e-3 / steps

        heur = kx.make_override(no_table=1)
        run(heur, sets[0])
        torch.cuda.synchronize()
        want = sets[0][4].float().clone()
        est = block(heur, 3)
        steps = int(max(5, min(300, block_s / max(est, 1e-7))))
        heur_t = est

        def duel(a, b):
            """median time of a and b over interleaved blocks"""
            ta, tb = [], []
            for _ in range(rounds):
                time.sleep(0.1)
                ta.append(block(a, steps))
                tb.append(block(b, steps))
            return statistics.median(ta), statistics.median(tb)

        best_ov, best_fields, best_t = heur, None, None
        for fields in candidates(M, N, K, kx):
            ov = kx.make_override(no_table=1, **fields)
            try:
                kx.kx_plan_query(M, N, K, ov=ov)
            except kx.KxError:
                continue
            sets[0][4].fill_(float("nan"))
            run(ov, sets[0])
            code, _ = kx.kx_last_device_status()
            got = sets[0][4].float()
            ok = code == 0 and bool(((got - want).abs() <= ATOL + RTOL * want.abs()).all())
            if not ok:
                if verbose:
                    print(f"[tune] {name}: REJECT {fields} (output differs from the heuristic plan's)", flush=True)
                continue
            t_inc, t_new = duel(best_ov, ov)
            if best_t is None:
                heur_t = t_inc
            if t_new < t_inc * (1.0 - margin):
                best_ov, best_fields, best_t = ov, fields, t_new
                if verbose:
                    print(f"[tune] {name}: KEEP {fields} {t_new*1e6:.1f} us vs {t_inc*1e6:.1f} us", flush=True)
            elif best_t is None:
                best_t = t_inc
        rec = {"name": name, "M": M, "N": N, "K": K, "heuristic_us": heur_t * 1e6,
               "best_us": (best_t or heur_t) * 1e6, "best": best_fields}
        report.append(rec)
        if best_fields is not None:
            lo, hi = m_bucket(M)
            entries.append((lo, hi, N, K, best_fields, name, heur_t, best_t))
        if verbose:
            print(f"[tune] {name}: heuristic {heur_t*1e6:.1f} us -> best {rec['best_us']:.1f} us {best_fields}", flush=True)
        del sets
        torch.cuda.empty_cache()
    return entries, report


def write_table(entries, path, margin):
    seen, lines = set(), []
    for lo, hi, N, K, fields, name, t0, t1 in entries:
        key = (lo, hi, N, K)
        if key in seen:
            continue
        seen.add(key)
        vals = ", ".join(str(int(fields.get(f, 0))) for f in FIELDS)
        lines.append(f"{{{lo}, {hi}, {N}, {K}, {vals}}},   // {name}: {t0*1e6:.1f} -> {t1*1e6:.1f} us")
    with open(path, "w") as f:
        f.write("// Measured plan table: {M_lo, M_hi, N, K, " + ", ".join(FIELDS) + "}\n")
        f.write("// Written by `python -m paper_2608_17071_b200.tune` on a B200 (keep margin "
                f"{margin:.0%}); empty = heuristics only.\n")
        for ln in lines:
            f.write(ln + "\n")


def main():
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--out", default=os.path.join(HERE, "csrc", "kx_plan_table.inc"))
    ap.add_argument("--report", default=None, help="optional JSON report path")
    ap.add_argument("--margin", type=float, default=0.03)
    ap.add_argument("--rounds", type=int, default=3)
    ap.add_argument("--block-ms", type=float, default=20.0)
    args = ap.parse_args()
    entries, report = tune(args.margin, args.rounds, args.block_ms * 1e-3)
    write_table(entries, args.out, args.margin)
    if args.report:
        with open(args.report, "w") as f:
            json.dump(report, f, indent=1)
    print(f"[tune] wrote {len(entries)} entries to {args.out}")


if __name__ == "__main__":
    main()
