"""Throughput report over the benchmark configurations and the size / users / shape / format sweep.

    python -m paper_2203_09044_b200.sweep --configs 0,1,2,3 --sweep --out report.md

For every workload it runs CO3 iterations (co3_encode + co3_decode_aggregate) on seeded synthetic
GenNorm gradients and prints one markdown table row: milliseconds per steady-state iteration, GB/s
of fp32 gradient, the fused convert pass against its 13 B per user-element, the encode passes, the
decode-aggregate pass, and the code / container bits per element.  All times are CUDA-event times;
per-kernel times come from the library's own event pairs around each launch.  Nothing here touches
the CPU oracle: this is a measurement script, parity lives in tests/.

Cells whose gradients and memories alone would need more than --max-bytes of device memory are
listed as skipped (the largest sweep cell, 2^28 elements x 64 users, needs about 160 GiB).
"""
import argparse
import json
import os
import sys

import torch

from . import binding, inputs

L2_BYTES = 126e6
NOMINAL_HBM_GBS = 8000.0
FORMATS = ((1, 2), (3, 2), (4, 3))                      # E1M2 (fp4), E3M2 (fp6), E4M3 (fp8)


def measured_hbm_gbs():
    """Measured copy bandwidth of this machine's GPUs if the file is there, else the fallback figure."""
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def device_bytes_needed(wl, pool, tile_users=None):
    """Gradients (pool copies, or two tiles of users), memory, symbols, worst-case payload and the average."""
    ud = wl.n_users * wl.d
    grads = 4 * ud * pool if tile_users is None else 2 * 4 * tile_users * wl.d
    return grads + 4 * ud + ud + 2 * ud + 4 * wl.d


def measure_tiled(wl, iters, warm, tile_users, rule=0):
    """As measure(), for a workload whose gradients do not fit at once: every iteration is fed in
    tiles of users, each drawn on the device right before it is consumed.  Only the library calls are
    timed (event pairs around each); drawing the gradients is not."""
    wl.align_rows()
    U, d = wl.n_users, wl.d
    plan = binding.Plan(d, U, wl.exp_bits, wl.mant_bits, wl.seg_offsets, gamma=wl.gamma, ld=wl.ld, bias_rule=rule)
    out = plan.alloc_outputs()
    residual = torch.zeros((U, plan.ld), dtype=torch.float32, device="cuda")
    pairs = []

    def around(after):
        ev = torch.cuda.Event(enable_timing=True)
        ev.record()
        if after:
            pairs[-1].append(ev)
        else:
            pairs.append([ev])

    def run(t):
        del pairs[:]
        plan.encode_tiled(tile_users, lambda u0, n: wl.gradient(t, device="cuda", users=range(u0, u0 + n)),
                          residual, out, around_call=around)
        around(False)
        plan.decode_aggregate(out)
        around(True)
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in pairs)

    first_ms = run(0)
    for t in range(1, warm):
        run(t)
    plan.profile_enable(None, max_records=(2 * (U // tile_users + 2)) * iters + 8)
    ms = sum(run(warm + t) for t in range(iters)) / iters
    prof = {k: v[0] / iters for k, v in plan.profile_collect().items() if v[1]}
    plan.profile_enable([], 0)
    flags, _ = plan.status(clear=True)
    code_bits = float(out["user_bits"].sum().item()) / (U * d)
    container_bits = (32.0 * float(out["chunk_off"][:, -1].sum().item()) + 16.0 * U * plan.n_sub
                      + 32.0 * U * (plan.n_chunks + 1) + 32.0 * plan.S) / (U * d)
    err2 = float(sum((residual[u, :d].double() ** 2).sum().item() for u in range(U)))
    s2 = sum(plan.get_fit(l)[4] for l in range(plan.S))
    ent_bits, emp_bits, model_bits = code_mismatch(plan, out)
    res = dict(rel_mse=err2 / s2 if s2 > 0 else 0.0, ent_bits=ent_bits, emp_bits=emp_bits, model_bits=model_bits,
               name=wl.name, d=d, U=U, S=plan.S, fmt="E%dM%d" % (wl.exp_bits, wl.mant_bits), beta=wl.beta,
               ms=ms, first_ms=first_ms, gbs=4.0 * U * d / (ms * 1e-3) / 1e9, convert_ms=prof.get("convert", 0.0),
               encode_ms=prof.get("enc_pack", 0.0), fit_ms=prof.get("fit", 0.0), decode_ms=prof.get("decode", 0.0),
               code_bits=code_bits, container_bits=container_bits, flags=flags, l2_resident=False,
               tiled=tile_users)
    plan.close()
    del out, residual
    torch.cuda.empty_cache()
    return res


def huffman_cost(counts):
    """Total code bits of an (unrestricted-depth) Huffman code built from these symbol counts: the
    sum of the weights of all internal nodes.  Symbols that do not occur get no codeword."""
    import heapq
    h = [int(c) for c in counts if c > 0]
    if len(h) <= 1:
        return float(sum(h))                            # one symbol still needs one bit each
    heapq.heapify(h)
    total = 0
    while len(h) > 1:
        a, b = heapq.heappop(h), heapq.heappop(h)
        total += a + b
        heapq.heappush(h, a + b)
    return float(total)


def code_mismatch(plan, out):
    """Per element, pooled over segments and users, for the last encoded iteration: the entropy of
    the symbol histogram, the bits of a Huffman code built from that histogram (what an
    empirical-histogram variant would spend, its code table not counted), and the bits of the model
    code actually used (histogram x code lengths of the rows the headers select)."""
    import numpy as np
    hist = plan.debug_hist().astype(np.float64)         # [S][nsym]
    if plan.bias_mode == binding.CODE_EMPIRICAL:
        lens = out["code_lens"].cpu().numpy()           # the code is the length table itself
    else:
        lens, _ = plan.debug_code(out["hdr"])           # [S][nsym]
    n = hist.sum()
    ent = 0.0
    for row in hist:
        t = row.sum()
        p = row[row > 0] / t if t > 0 else row[:0]
        ent += -float((p * np.log2(p)).sum()) * t
    emp = sum(huffman_cost(row) for row in hist)
    model = float((hist * lens).sum())
    return ent / n, emp / n, model / n


def measure(wl, iters, warm, pool, rule=0, mode=None):
    """Run warm + iters iterations of one workload; returns a dict of figures."""
    wl.align_rows()
    U, d = wl.n_users, wl.d
    plan = binding.Plan(d, U, wl.exp_bits, wl.mant_bits, wl.seg_offsets, gamma=wl.gamma,
                        bias_mode=binding.BIAS_LAGGED if mode is None else mode, ld=wl.ld, bias_rule=rule)
    out = plan.alloc_outputs()
    residual = torch.zeros((U, plan.ld), dtype=torch.float32, device="cuda")
    grads = [wl.gradient(t, device="cuda") for t in range(pool)]
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def step(t):
        plan.encode(grads[t % pool], residual, out)
        plan.decode_aggregate(out)

    e0.record()
    step(0)                                             # t = 0: includes the bootstrap statistics pass
    e1.record()
    torch.cuda.synchronize()
    first_ms = e0.elapsed_time(e1)
    for t in range(1, warm):
        step(t)
    torch.cuda.synchronize()
    e0.record()
    for t in range(iters):
        step(warm + t)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    # the per-kernel breakdown comes from a second set of iterations: an event pair around every
    # launch costs a few microseconds, which the figure above should not carry
    plan.profile_enable(None, max_records=2 * iters + 8)
    for t in range(iters):
        step(warm + iters + t)
    torch.cuda.synchronize()
    prof = {k: v[0] / iters for k, v in plan.profile_collect().items() if v[1]}
    plan.profile_enable([], 0)
    # a steady-state iteration has no host decision in it: the same steps replayed from one CUDA graph
    graph_ms = None
    if mode in (None, binding.BIAS_LAGGED, binding.BIAS_CURRENT, binding.CODE_LAGGED):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, capture_error_mode="thread_local"):
            for t in range(pool):
                step(t)
        graph.replay()
        torch.cuda.synchronize()
        reps = max(1, (iters + pool - 1) // pool)
        e0.record()
        for _ in range(reps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        graph_ms = e0.elapsed_time(e1) / (reps * pool)
        del graph
    flags, nonfinite = plan.status(clear=True)
    code_bits = float(out["user_bits"].sum().item()) / (U * d)
    container_bits = (32.0 * float(out["chunk_off"][:, -1].sum().item()) + 16.0 * U * plan.n_sub
                      + 32.0 * U * (plan.n_chunks + 1) + 32.0 * plan.S) / (U * d)
    # realised relative conversion error of the last iteration: the memory is a - Q(a) exactly
    err2 = float((residual[:, :d].double() ** 2).sum().item())
    s2 = sum(plan.get_fit(l)[4] for l in range(plan.S))
    ent_bits, emp_bits, model_bits = code_mismatch(plan, out)
    res = dict(rel_mse=err2 / s2 if s2 > 0 else 0.0, ent_bits=ent_bits, emp_bits=emp_bits, model_bits=model_bits,
               name=wl.name, d=d, U=U, S=plan.S, fmt="E%dM%d" % (wl.exp_bits, wl.mant_bits), beta=wl.beta,
               ms=ms, first_ms=first_ms, gbs=4.0 * U * d / (ms * 1e-3) / 1e9,
               convert_ms=prof.get("convert", 0.0),
               encode_ms=prof.get("enc_scan", 0.0) + prof.get("enc_pack", 0.0)
               + prof.get("code_enc", 0.0),
               fit_ms=prof.get("fit", 0.0), decode_ms=prof.get("decode", 0.0) + prof.get("code_dec", 0.0),
               code_bits=code_bits, container_bits=container_bits, flags=flags,
               l2_resident=8.0 * U * d * pool < L2_BYTES, graph_ms=graph_ms)
    plan.close()
    del out, residual, grads
    torch.cuda.empty_cache()
    return res


def gamma_sweep(wl, gammas, iters):
    """Memory decay sweep (the quantity of the paper's Fig. 3 on synthetic streams): L1 norm of the
    memory over L1 norm of the gradient after every iteration, per gamma, with the model update fused
    into the decode (weights start at zero, step -0.01).  Returns {gamma: [ratio per iteration]}."""
    U, d = wl.n_users, wl.d
    out_rows = {}
    for gamma in gammas:
        plan = binding.Plan(d, U, wl.exp_bits, wl.mant_bits, wl.seg_offsets, gamma=gamma, ld=wl.ld)
        out = plan.alloc_outputs()
        residual = torch.zeros((U, plan.ld), dtype=torch.float32, device="cuda")
        weights = torch.zeros(d, dtype=torch.float32, device="cuda")
        ratios = []
        for t in range(iters):
            g = wl.gradient(t, device="cuda")
            plan.encode(g, residual, out)
            plan.decode_aggregate_update(out, weights, -0.01)
            ratios.append(float(residual[:, :d].abs().sum().item() / g[:, :d].abs().sum().item()))
        assert plan.status()[0] == 0
        plan.close()
        out_rows[gamma] = ratios
    return out_rows


HEADER = ("| workload | d | U | format | beta | ms/iter | GB/s fp32 in | convert us | convert GB/s (13 B) | % of {peak:.0f} "
          "| % of 8000 | encode us | decode us | decode+encode GB/s (payload+symbols+avg) | code b/el | container b/el | t=0 ms | rel. sq. error | entropy b/el | Huffman(histogram) b/el | note |\n"
          "|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|")


def row(r, peak):
    ud = r["U"] * r["d"]
    conv_gbs = 13.0 * ud / (r["convert_ms"] * 1e-3) / 1e9 if r["convert_ms"] else 0.0
    # encode + decode algorithmic bytes: symbols read twice, payload written and read, average written
    ed_bytes = 2.0 * ud + 2.0 * r["code_bits"] / 8.0 * ud + 4.0 * r["d"]
    ed_ms = r["encode_ms"] + r["decode_ms"]
    ed_gbs = ed_bytes / (ed_ms * 1e-3) / 1e9 if ed_ms else 0.0
    note = []
    if r["l2_resident"]:
        note.append("inputs fit L2, launch-bound")
    if r.get("graph_ms"):
        note.append("%.4f ms from a CUDA graph" % r["graph_ms"])
    if r["flags"]:
        note.append("flags=%d" % r["flags"])
    if r.get("tiled"):
        note.append("gradients fed in tiles of %d users (co3_tiled_*), drawn per tile, drawing not timed" % r["tiled"])
    return ("| %s | %d | %d | %s | %.1f | %.4f | %.1f | %.1f | %.0f | %.1f | %.1f | %.1f | %.1f | %.0f | %.3f | %.3f | %.3f | %.3e | %.3f | %.3f | %s |"
            % (r["name"], r["d"], r["U"], r["fmt"], r["beta"], r["ms"], r["gbs"], r["convert_ms"] * 1e3, conv_gbs,
               100.0 * conv_gbs / peak, 100.0 * conv_gbs / NOMINAL_HBM_GBS, r["encode_ms"] * 1e3,
               r["decode_ms"] * 1e3, ed_gbs, r["code_bits"], r["container_bits"], r["first_ms"],
               r.get("rel_mse", 0.0), r.get("ent_bits", 0.0), r.get("emp_bits", 0.0), "; ".join(note)))


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--configs", default="0,1,2,3", help="comma list of benchmark configurations (empty: none)")
    ap.add_argument("--sweep", action="store_true", help="also run the 108-cell sweep")
    ap.add_argument("--iters", type=int, default=5, help="timed steady-state iterations per workload")
    ap.add_argument("--warm", type=int, default=3, help="untimed iterations before them (>= 1)")
    ap.add_argument("--max-bytes", type=float, default=60e9, help="skip workloads needing more device memory")
    ap.add_argument("--tile-users", type=int, default=0,
                    help="workloads over --max-bytes: feed the gradients in tiles of this many users if that "
                         "fits --max-tiled-bytes (0: skip them)")
    ap.add_argument("--max-tiled-bytes", type=float, default=150e9)
    ap.add_argument("--mode", default="lagged", choices=["lagged", "current", "code-lagged", "empirical"],
                    help="bias/code mode of the plans (default: lagged bias, the benchmark configuration)")
    ap.add_argument("--rule", default="poly", choices=["poly", "opt"],
                    help="bias rule: the paper's polynomial (default) or the L2-optimal integer bias")
    ap.add_argument("--gamma-sweep", action="store_true",
                    help="instead: memory L1 / gradient L1 per iteration for gamma in {0, 0.1, 0.5, 0.9, 1} on "
                         "configuration 1's layers in the 4-bit format")
    ap.add_argument("--filter", default=None, help="run only workloads whose name contains this text")
    ap.add_argument("--out", default=None, help="also write the table to this file")
    args = ap.parse_args(argv)
    binding.lib()                                       # no CUDA library: raise, never fall back
    if args.gamma_sweep:
        wl = inputs.workload(1).align_rows()
        wl.exp_bits, wl.mant_bits = 1, 2                # the paper's 4-bit format, as in its gamma experiment
        rows = gamma_sweep(wl, (0.0, 0.1, 0.5, 0.9, 1.0), 12)
        lines = ["| gamma | " + " | ".join("t=%d" % t for t in range(12)) + " |", "|---|" + "---|" * 12]
        for gm, r in rows.items():
            lines.append("| %.1f | " % gm + " | ".join("%.4f" % x for x in r) + " |")
        text = "\n".join(lines) + "\n"
        if args.out:
            with open(args.out, "w") as f:
                f.write(text)
        sys.stdout.write(text)
        return 0
    peak, src = measured_hbm_gbs()
    lines = ["Peak used for the convert column: %.1f GB/s (%s copy bandwidth); nominal 8000 GB/s beside it." % (peak, src),
             "", HEADER.format(peak=peak)]
    todo = [inputs.workload(int(i)) for i in args.configs.split(",") if i != ""]
    if args.sweep:
        for d_log in (16, 20, 24, 28):
            for users in (1, 8, 64):
                for beta in (0.5, 1.0, 2.0):
                    for e, m in FORMATS:
                        todo.append(inputs.sweep_cell(1 << d_log, users, beta, e, m))
    if args.filter:
        todo = [wl for wl in todo if args.filter in wl.name]
    for wl in todo:
        pool = 2 if device_bytes_needed(wl, 2) <= args.max_bytes else 1
        if device_bytes_needed(wl, pool) > args.max_bytes and args.tile_users > 0 and args.mode == "lagged" \
                and device_bytes_needed(wl, 1, args.tile_users) <= args.max_tiled_bytes:
            r = measure_tiled(wl, args.iters, max(args.warm, 1), args.tile_users,
                              binding.RULE_OPT if args.rule == "opt" else binding.RULE_POLY)
            lines.append(row(r, peak))
            print(lines[-1], flush=True)
            continue
        if device_bytes_needed(wl, pool) > args.max_bytes:
            lines.append("| %s | %d | %d | E%dM%d | %.1f | skipped: needs %.0f GB of device memory | | | | | | | | | | | | | | |"
                         % (wl.name, wl.d, wl.n_users, wl.exp_bits, wl.mant_bits, wl.beta,
                            device_bytes_needed(wl, 1) / 1e9))
            continue
        mode = {"lagged": binding.BIAS_LAGGED, "current": binding.BIAS_CURRENT, "code-lagged": binding.CODE_LAGGED,
                "empirical": binding.CODE_EMPIRICAL}[args.mode]
        r = measure(wl, args.iters, max(args.warm, 1), pool,
                    binding.RULE_OPT if args.rule == "opt" else binding.RULE_POLY, mode)
        lines.append(row(r, peak))
        print(lines[-1], flush=True)
    text = "\n".join(lines) + "\n"
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)
    else:
        sys.stdout.write(text)
    return 0


if __name__ == "__main__":
    sys.exit(main())
