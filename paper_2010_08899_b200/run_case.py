"""Run one entry point of the library a few times on seeded synthetic data.

A small command-line driver for profiling and quick timing of a single kernel at a chosen size:

    python -m paper_2010_08899_b200.run_case compress --n 268435456 --iters 3
    python -m paper_2010_08899_b200.run_case select   --n 268435456 --k 26844
    python -m paper_2010_08899_b200.run_case mp_fwd   --rows 16384 --d 4096 --k 205 --dtype bf16
    python -m paper_2010_08899_b200.run_case mp_bwd   --rows 16384 --d 4096 --k 205 --dtype bf16
    python -m paper_2010_08899_b200.run_case select_compress --n 268435456   (threshold life-span L = 1)
    python -m paper_2010_08899_b200.run_case decompress --n 268435456
    python -m paper_2010_08899_b200.run_case mp_unpack --rows 16384 --d 4096 --k 205 --dtype bf16
    python -m paper_2010_08899_b200.run_case select_multi --n 268435456          (75 / 90 / 95 % sparsity)
    python -m paper_2010_08899_b200.run_case threshold_mean --rows 16384 --d 4096 --dtype bf16
    python -m paper_2010_08899_b200.run_case mp_fwd_sweep --dtype bf16    (a table: row widths x sparsity levels)
    python -m paper_2010_08899_b200.run_case dp_sweep                     (a table: vector sizes x densities)
    python -m paper_2010_08899_b200.run_case receiver_sweep               (backward pack, unpack, decompress over shapes)

It prints the mean device time per call (CUDA events) and the algorithmic GB/s.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as B
from . import inputs


def mp_fwd_sweep(args, dev, stream):
    """The forward pack over row widths and sparsity levels, about 128 MiB of activations per cell (the generator of
    the bench: ReLU of a Gaussian with log-normal column scales), `--iters` launches back to back after a warm-up
    round; prints the algorithmic TB/s (input + k (2 + s) bytes per row)."""
    dt = torch.float32 if args.dtype == "f32" else torch.bfloat16
    es = 4 if args.dtype == "f32" else 2
    widths = [64, 128, 192, 256, 320, 384, 512, 768, 1024, 1536, 2048, 3072, 4096, 6144, 8192, 12288, 16384, 32768]
    fracs = [0.02, 0.05, 0.10, 0.25, 0.375, 0.5]
    print("d      " + "".join(f"{f * 100:>9.1f}%" for f in fracs) + "   TB/s algorithmic, k = fraction of d")
    for d in widths:
        rows = max(64, (128 << 20) // (d * es))
        x = inputs.mp_activations(rows, d, 7 + d, dtype=dt, device=dev, col_scale_seed=8 + d)
        k_max = max(1, int(d * max(fracs)))
        cols = torch.empty(rows * k_max, dtype=torch.int16, device=dev)       # sized for the largest k of the row
        vals = torch.empty(rows * k_max, dtype=dt, device=dev)
        line = f"{d:<7d}"
        for f in fracs:
            k = max(1, int(d * f))
            for phase in range(2):
                a = torch.cuda.Event(enable_timing=True)
                b = torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for _ in range(args.iters):
                    B.dct_mp_topk_pack_fwd(x, rows, d, d, k, cols[: rows * k], vals[: rows * k], None, None, None, stream)
                b.record(stream)
                b.synchronize()
            ms = a.elapsed_time(b) / args.iters
            line += f"{(rows * d * es + rows * k * (2 + es)) / (ms * 1e-3) / 1e12:10.2f}"
        print(line, flush=True)
        del x, cols, vals


def dp_sweep(args, dev, stream):
    """DCT-DP over vector sizes and densities k / n: the select, then `--iters` compress iterations with that
    threshold (the error carried from one to the next, a fresh gradient each time from two shifted buffers), and the
    one-call L = 1 iteration.  Prints ms per call and the algorithmic TB/s (select: 4 B per element read once;
    compress and L = 1: 12 B per element + 8 B per survivor)."""
    sizes = [1 << 16, 1 << 20, 1 << 22, 1 << 24, 1 << 25, 1 << 26, 1 << 28, 1 << 30]
    densities = [1e-4, 1e-3, 1e-2, 0.05, 0.25]
    print("n         density        k   select ms (TB/s)   compress ms (TB/s)   L=1 ms (TB/s)")
    for n in sizes:
        slack = 64
        g = [inputs.dp_mixture(n + slack, 11 + j, dev) for j in range(2)]
        e = torch.zeros(n, device=dev)
        tau = torch.zeros(1, device=dev)
        idx = torch.empty(n, dtype=torch.int32, device=dev)                    # capacity n: nothing is cut off
        val = torch.empty(n, device=dev)
        res = B.new_result(dev)
        ws_s = B.new_workspace(B.dct_threshold_select_workspace_bytes(n), dev)
        ws_c = B.new_workspace(B.dct_dp_compress_workspace_bytes(n), dev)
        ws_l = B.new_workspace(B.dct_dp_select_compress_workspace_bytes(n), dev)
        fresh = lambda i: g[i % 2][4 * (i // 2): 4 * (i // 2) + n]

        def timed(call, reps):
            for phase in range(2):
                a = torch.cuda.Event(enable_timing=True)
                b = torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for i in range(reps):
                    call(i)
                b.record(stream)
                b.synchronize()
            return a.elapsed_time(b) / reps

        for dens in densities:
            k = max(1, int(n * dens))
            ms_s = timed(lambda i: B.dct_threshold_select(fresh(i), None, n, k, tau, res, ws_s, stream), args.iters)
            B.dct_threshold_select(fresh(0), None, n, k, tau, res, ws_s, stream)
            e.zero_()
            ms_c = timed(lambda i: B.dct_dp_compress(fresh(i), e, n, tau, None, idx, val, n, res, ws_c, stream), args.iters)
            surv = B.read_result(res).count
            e.zero_()
            ms_l = timed(lambda i: B.dct_dp_select_compress(fresh(i), e, n, k, tau, idx, val, n, res, ws_l, stream), args.iters)
            tb = lambda bytes_, ms: bytes_ / (ms * 1e-3) / 1e12
            print(f"2^{n.bit_length() - 1:<3d} {dens:10.4f} {k:12d}   {ms_s:8.4f} ({tb(4 * n, ms_s):5.2f})"
                  f"   {ms_c:8.4f} ({tb(12 * n + 8 * surv, ms_c):5.2f})   {ms_l:8.4f} ({tb(12 * n + 8 * k, ms_l):5.2f})", flush=True)
        del g, e, idx, val, ws_s, ws_c, ws_l


def receiver_sweep(args, dev, stream):
    """The backward pack and the receiver side over shapes: `dct_mp_pack_bwd` and `dct_mp_unpack` for both dtypes, row
    widths from 64 to 32768 columns and k = 1 %, 5 % and 25 % of the row (192 MiB of matrix per cell; the forward pack
    beside them), then `dct_dp_decompress` (overwriting and accumulating) at N = 2^28 over survivor densities.  ms per
    call and TB/s: forward and unpack count the dense matrix + the packed entries, the backward pack the dense matrix
    (what reaches DRAM), decompress 4 B (accumulating: 8 B) per element + 8 B per survivor."""
    def timed(call, reps):
        for phase in range(2):
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i in range(reps):
                call(i)
            b.record(stream)
            b.synchronize()
        return a.elapsed_time(b) / reps
    print("dtype      d     k     rows |  fwd ms (TB/s) |  bwd ms (TB/s) | unpack ms (TB/s)")
    for dt, es in ((torch.bfloat16, 2), (torch.float32, 4)):
        for d in (64, 128, 256, 512, 1024, 2048, 4096, 8192, 16384, 32768):
            rows = max(256, (192 << 20) // (d * es))
            kmax = max(1, d // 4)
            x = [inputs.mp_activations(rows, d, 410 + j, dtype=dt, device=dev, col_scale_seed=400) for j in range(2)]
            gx = [inputs.mp_gradients(rows, d, 420 + j, dtype=dt, device=dev) for j in range(2)]
            cols = torch.empty(rows * kmax, dtype=torch.int16, device=dev)
            vals = torch.empty(rows * kmax, dtype=dt, device=dev)
            gv = torch.empty(rows * kmax, dtype=dt, device=dev)
            dense = [torch.empty(rows, d, dtype=dt, device=dev) for _ in range(2)]
            for k in sorted({max(1, d // 100), max(1, d // 20), max(1, d // 4)}):
                f = timed(lambda i: B.dct_mp_topk_pack_fwd(x[i % 2], rows, d, d, k, cols, vals, None, None, None, stream), args.iters)
                B.dct_mp_topk_pack_fwd(x[0], rows, d, d, k, cols, vals, None, None, None, stream)
                bw = timed(lambda i: B.dct_mp_pack_bwd(gx[i % 2], rows, d, d, k, cols, gv, None, stream), args.iters)
                u = timed(lambda i: B.dct_mp_unpack(cols, vals, rows, d, d, k, dense[i % 2], None, stream), args.iters)
                nb, pk = rows * d * es, rows * k * (2 + es)
                print(f"{'bf16' if es == 2 else 'f32 '} {d:6d} {k:5d} {rows:8d} | {f:7.4f} ({(nb + pk) / f / 1e9:5.2f}) | "
                      f"{bw:7.4f} ({nb / bw / 1e9:5.2f}) | {u:7.4f} ({(nb + pk) / u / 1e9:5.2f})", flush=True)
            del x, gx, cols, vals, gv, dense
    n = 1 << 28
    print(f"decompress, N = 2^28: survivors | overwrite ms (TB/s) | accumulate ms (TB/s)")
    g = inputs.dp_mixture(n, 7, dev)
    e = torch.zeros(n, device=dev)
    tau, res, res2 = torch.zeros(1, device=dev), B.new_result(dev), B.new_result(dev)
    ws_s = B.new_workspace(B.dct_threshold_select_workspace_bytes(n), dev)
    ws_c = B.new_workspace(B.dct_dp_compress_workspace_bytes(n), dev)
    cap = n // 4 + 1024
    idx = torch.empty(cap, dtype=torch.int32, device=dev)
    val = torch.empty(cap, device=dev)
    dense = torch.empty(n, device=dev)
    for dens in (1e-4, 1e-3, 1e-2, 0.05, 0.25):
        B.dct_threshold_select(g, None, n, int(n * dens), tau, res, ws_s, stream)
        e.zero_()
        B.dct_dp_compress(g, e, n, tau, None, idx, val, cap, res, ws_c, stream)
        cnt = B.read_result(res).count
        packed = res.clone()
        ms = timed(lambda i: B.dct_dp_decompress(idx, val, packed, cap, dense, n, False, res2, stream), args.iters)
        ms_a = timed(lambda i: B.dct_dp_decompress(idx, val, packed, cap, dense, n, True, res2, stream), args.iters)
        print(f"{cnt:10d} ({100 * dens:g} %) | {ms:7.4f} ({(4 * n + 8 * cnt) / ms / 1e9:5.2f}) | "
              f"{ms_a:7.4f} ({(8 * n + 8 * cnt) / ms_a / 1e9:5.2f})", flush=True)


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("entry", choices=["select", "compress", "select_compress", "compress_layers", "decompress", "mp_fwd", "mp_bwd", "mp_unpack",
                                     "select_multi", "threshold_mean", "mp_fwd_sweep", "dp_sweep", "receiver_sweep"])
    ap.add_argument("--n", type=int, default=1 << 28)
    ap.add_argument("--k", type=int, default=0, help="survivor target (default: 0.01 %% of n, or 5 %% of d)")
    ap.add_argument("--rows", type=int, default=16384)
    ap.add_argument("--d", type=int, default=4096)
    ap.add_argument("--dtype", choices=["f32", "bf16"], default="bf16")
    ap.add_argument("--dist", choices=["mixture", "gaussian", "dlrm"], default="mixture")
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    ap.add_argument("--l2-fetch", type=int, default=0, choices=[0, 32, 64, 128],
                    help="set this process's cudaLimitMaxL2FetchGranularity hint (bytes) before anything runs")
    ap.add_argument("--back-to-back", action="store_true",
                    help="time all iterations between one pair of events (launch gaps overlap, as in a training loop)")
    args = ap.parse_args()

    dev = "cuda"
    if args.l2_fetch:
        # a hint of this process's CUDA context (it dies with the process; no setting of the GPU changes)
        import ctypes
        import glob
        import os
        torch.cuda.init()
        torch.zeros(1, device=dev)                                            # the primary context exists
        found = glob.glob(os.path.join(os.path.dirname(torch.__file__), "..", "nvidia", "cuda_runtime", "lib", "libcudart.so*"))
        rt = ctypes.CDLL(found[0] if found else "libcudart.so")
        rc = rt.cudaDeviceSetLimit(5, ctypes.c_size_t(args.l2_fetch))         # 5 = cudaLimitMaxL2FetchGranularity
        got = ctypes.c_size_t(0)
        rt.cudaDeviceGetLimit(ctypes.byref(got), 5)
        print(f"cudaLimitMaxL2FetchGranularity <- {args.l2_fetch} B: return code {rc}, now {got.value} B")
    stream = torch.cuda.current_stream()
    reset = lambda: None
    if args.entry == "mp_fwd_sweep":
        return mp_fwd_sweep(args, dev, stream)
    if args.entry == "dp_sweep":
        return dp_sweep(args, dev, stream)
    if args.entry == "receiver_sweep":
        return receiver_sweep(args, dev, stream)
    gen = {"mixture": inputs.dp_mixture, "gaussian": inputs.dp_gaussian, "dlrm": inputs.dp_dlrm_like}[args.dist]

    if args.entry == "compress_layers":
        # the vector of --n elements cut into DLRM-like dense layers, each with its own threshold and error:
        # one batched call against one dct_dp_compress call per layer
        sizes, total = [], 0
        while total < args.n:
            for fo, fi in inputs.DLRM_LIKE_LAYERS:
                if total < args.n:
                    sizes.append(min(fo * fi, args.n - total))
                    total += sizes[-1]
        g_all = inputs.dp_dlrm_like(args.n, 301, dev)
        e_all = torch.zeros(args.n, device=dev)
        layers, sel_layers, off = [], [], 0
        for m in sizes:
            cap = max(m // 16, 64)
            tau = torch.zeros(1, device=dev)
            sel_layers.append(dict(grad=g_all[off:off + m], residual=None, n=m, k=B.k_from_density(m, 1, 1000),
                                   tau_out=tau, result=B.new_result(dev)))
            layers.append(dict(grad=g_all[off:off + m], residual=e_all[off:off + m], n=m, tau=tau, tie_budget=None,
                               idx_out=torch.empty(cap, dtype=torch.int32, device=dev),
                               val_out=torch.empty(cap, device=dev), capacity=cap, result=B.new_result(dev)))
            off += m
        # the thresholds of all layers: one batched call against one dct_threshold_select call per layer
        ws_sb = B.new_workspace(B.dct_threshold_select_batched_workspace_bytes(len(sizes)), dev)
        ws_s1 = B.new_workspace(B.dct_threshold_select_workspace_bytes(max(sizes)), dev)
        sel_table = B.dct_select_layer_table(sel_layers)
        sel_variants = {
            f"select, batched ({len(sizes)} layers, one call)": lambda: B.dct_threshold_select_batched(sel_table, ws_sb),
            f"select, one call per layer ({len(sizes)} calls)": lambda: [B.dct_threshold_select(
                a["grad"], None, a["n"], a["k"], a["tau_out"], a["result"], ws_s1) for a in sel_layers],
        }
        for name, fn in sel_variants.items():
            for phase in range(2):
                a = torch.cuda.Event(enable_timing=True)
                b = torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                b.synchronize()
            ms = a.elapsed_time(b)
            print(f"compress_layers, {name}: {ms:.4f} ms, {4 * args.n / ms / 1e6:.1f} GB/s at the 4 B floor")
        ws_b = B.new_workspace(B.dct_dp_compress_batched_workspace_bytes(sizes), dev)
        ws_1 = B.new_workspace(B.dct_dp_compress_workspace_bytes(max(sizes)), dev)
        table = B.dct_dp_layer_table(layers)      # marshalled once, as a trainer would
        variants = {
            f"batched ({len(sizes)} layers, one call)": lambda: B.dct_dp_compress_batched(table, ws_b),
            f"one call per layer ({len(sizes)} calls)": lambda: [B.dct_dp_compress(
                a["grad"], a["residual"], a["n"], a["tau"], None, a["idx_out"], a["val_out"], a["capacity"],
                a["result"], ws_1) for a in layers],
        }
        for name, fn in variants.items():
            for phase in range(2):
                e_all.zero_()
                a = torch.cuda.Event(enable_timing=True)
                b = torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                b.synchronize()
            ms = a.elapsed_time(b)
            print(f"compress_layers, {name}: {ms:.4f} ms, {12 * args.n / ms / 1e6:.1f} GB/s algorithmic")
        return

    if args.entry == "select_multi":
        # the paper's three sparsity levels (75 / 90 / 95 %) out of one set of passes
        n = args.n
        ks = [B.k_from_sparsity(n, 75, 100), B.k_from_sparsity(n, 90, 100), B.k_from_sparsity(n, 95, 100)]
        g = [gen(n, 501 + j, dev) for j in range(2)]
        taus = torch.zeros(len(ks), device=dev)
        res = torch.zeros(5 * len(ks), dtype=torch.int64, device=dev)
        ws = B.new_workspace(B.dct_threshold_select_multi_workspace_bytes(n, len(ks)), dev)
        call = lambda i: B.dct_threshold_select_multi(g[i % 2], None, n, ks, taus, res, ws)
        nbytes = 4 * n
    elif args.entry == "threshold_mean":
        rows, d = args.rows, args.d
        dt = torch.float32 if args.dtype == "f32" else torch.bfloat16
        es = 4 if args.dtype == "f32" else 2
        ks = [B.k_from_sparsity(d, 75, 100), B.k_from_sparsity(d, 90, 100), B.k_from_sparsity(d, 95, 100)]
        x = [inputs.mp_activations(rows, d, 410 + j, dtype=dt, device=dev, col_scale_seed=400) for j in range(2)]
        mean = torch.zeros(len(ks), dtype=torch.float64, device=dev)
        tau_rows = torch.zeros(len(ks) * rows, dtype=dt, device=dev)
        call = lambda i: B.dct_mp_threshold_mean(x[i % 2], rows, d, d, ks, mean, tau_rows)
        nbytes = rows * d * es
    elif args.entry == "select_compress":
        # select and compress the same vector every iteration (exactly k survivors); the error carries over
        n = args.n
        k = args.k or B.k_from_density(n, 1, 10_000)
        g = [gen(n, 501 + j, dev) for j in range(2)]
        e = torch.zeros(n, device=dev)
        cap = max(n // 64, 1024)
        idx = torch.empty(cap, dtype=torch.int32, device=dev)
        val = torch.empty(cap, device=dev)
        tau, res = torch.zeros(1, device=dev), B.new_result()
        ws = B.new_workspace(B.dct_dp_select_compress_workspace_bytes(n), dev)
        call = lambda i: B.dct_dp_select_compress(g[i % 2], e, n, k, tau, idx, val, cap, res, ws)
        nbytes = 12 * n
    elif args.entry in ("select", "compress", "decompress"):
        n = args.n
        k = args.k or B.k_from_density(n, 1, 10_000)
        g = [gen(n, 501 + j, dev) for j in range(2)]
        tau = torch.zeros(1, device=dev)
        res = B.new_result(dev)
        ws_s = B.new_workspace(B.dct_threshold_select_workspace_bytes(n), dev)
        B.dct_threshold_select(g[0], None, n, k, tau, res, ws_s)
        if args.entry == "select":
            call = lambda i: B.dct_threshold_select(g[i % 2], None, n, k, tau, res, ws_s)
            nbytes = 4 * n
        else:
            e = torch.zeros(n, device=dev)
            cap = min(n, max(n // 64, 1024, 2 * k))      # room for every survivor of a zero residual
            idx = torch.empty(cap, dtype=torch.int32, device=dev)
            val = torch.empty(cap, device=dev)
            ws_c = B.new_workspace(B.dct_dp_compress_workspace_bytes(n), dev)
            call = lambda i: B.dct_dp_compress(g[i % 2], e, n, tau, None, idx, val, cap, res, ws_c)
            reset = e.zero_          # every timed call starts from a zero residual (same survivor density)
            nbytes = 12 * n
            if args.entry == "decompress":
                call(0)
                count = B.read_result(res).count
                packed = res.clone()
                dense = torch.empty(n, device=dev)
                res2 = B.new_result(dev)
                call = lambda i: B.dct_dp_decompress(idx, val, packed, cap, dense, n, False, res2)
                reset = lambda: None
                nbytes = 4 * n + 8 * count       # clear the dense vector, read the packed pairs
    else:
        rows, d = args.rows, args.d
        k = args.k or B.k_from_sparsity(d, 95, 100)
        dt = torch.float32 if args.dtype == "f32" else torch.bfloat16
        es = 4 if args.dtype == "f32" else 2
        x = [inputs.mp_activations(rows, d, 410 + j, dtype=dt, device=dev, col_scale_seed=400) for j in range(2)]
        cols = torch.empty(rows * k, dtype=torch.int16, device=dev)
        vals = torch.empty(rows * k, dtype=dt, device=dev)
        tau_i = torch.empty(rows, dtype=dt, device=dev)
        B.dct_mp_topk_pack_fwd(x[0], rows, d, d, k, cols, vals)
        if args.entry == "mp_fwd":
            call = lambda i: B.dct_mp_topk_pack_fwd(x[i % 2], rows, d, d, k, cols, vals, None, tau_i)
            nbytes = rows * d * es + rows * k * (2 + es)
        elif args.entry == "mp_unpack":
            dense = [torch.empty(rows, d, dtype=dt, device=dev) for _ in range(2)]
            call = lambda i: B.dct_mp_unpack(cols, vals, rows, d, d, k, dense[i % 2])
            nbytes = rows * d * es + rows * k * (2 + es)
        else:
            gx = [inputs.mp_gradients(rows, d, 420 + j, dtype=dt, device=dev) for j in range(2)]
            gv = torch.empty(rows * k, dtype=dt, device=dev)
            call = lambda i: B.dct_mp_pack_bwd(gx[i % 2], rows, d, d, k, cols, gv)
            nbytes = rows * k * (2 + es) + rows * k * es

    for i in range(args.warmup):
        reset()
        call(i)
    torch.cuda.synchronize()
    if args.back_to_back:
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(args.iters):
            call(i)
        b.record(stream)
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / args.iters
        print(f"{args.entry}: {ms:.4f} ms per call back to back, {nbytes / ms / 1e6:.1f} GB/s algorithmic ({nbytes} B per call)")
        return
    pairs = []
    for i in range(args.iters):
        reset()
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        a.record(stream)
        call(i)
        b.record(stream)
        pairs.append((a, b))
    torch.cuda.synchronize()
    ms = sum(a.elapsed_time(b) for a, b in pairs) / args.iters
    print(f"{args.entry}: {ms:.4f} ms per call, {nbytes / ms / 1e6:.1f} GB/s algorithmic ({nbytes} B per call)")


if __name__ == "__main__":
    main()
