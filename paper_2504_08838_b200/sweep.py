"""Sparsity sweep on single matrices: sd2_spmm against cuBLAS dense bf16, cold HBM.

    python -m paper_2504_08838_b200.sweep [--sparsities 0.3,0.5,...] [--n 1,16,64] [--quick]

For every shape (M x K) of the sweep (3072x8192, 8192x3072, 2048x11008), sparsity and N, the
matrix is compressed once on the host and loaded R times, R chosen so that the R copies are
at least four times the L2 cache: a CUDA graph of R launches, one per copy, then reads every
copy from HBM.  The dense baseline is torch.matmul (cuBLAS, bf16 in, fp32 accumulate) on the
masked weight stored densely, with the same rotation and the same graph treatment.  Prints a
markdown table: microseconds per launch, GB/s over the compressed bytes, and the lowest
sparsity at which the sparse launch is faster than the dense one (linear interpolation).
"""

from __future__ import annotations

import argparse

import numpy as np

from . import binding as sd2
from . import synth


def time_graph(torch, fn, reps):
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        fn()
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            fn()
        for _ in range(3):
            g.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
        stream.synchronize()
    return e0.elapsed_time(e1) / reps * 1e3      # microseconds per graph


def main():
    import torch
    ap = argparse.ArgumentParser()
    ap.add_argument("--sparsities", default="0.3,0.4,0.5,0.6,0.66,0.7,0.75,0.8,0.9")
    ap.add_argument("--n", default="1,16,64")
    ap.add_argument("--quick", action="store_true", help="first shape only")
    args = ap.parse_args()
    sparsities = [float(s) for s in args.sparsities.split(",")]
    ns = [int(n) for n in args.n.split(",")]
    shapes = synth.SWEEP_SHAPES[:1] if args.quick else synth.SWEEP_SHAPES
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    print("| M x K | N | sparsity | B / kept weight | sparse us | sparse GB/s | dense us | dense / sparse |")
    print("|---|---|---|---|---|---|---|---|")
    for (M, K) in shapes:
        W = synth.normal_bf16(synth.stream_seed(5, 0, 0, synth.WHAT_W) + M, (M, K), 0.02)
        cross = {n: [] for n in ns}
        for sp in sparsities:
            mask = synth.bernoulli_mask(synth.stream_seed(5, 0, 0, synth.WHAT_MASK) + M + int(1000 * sp), (M, K), 1.0 - sp)
            blob = sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_AUTO, sd2.SD2_DTYPE_BF16)
            h0 = sd2.sd2_load_blob(blob)
            R = max(2, int(np.ceil(4.0 * l2 / h0.compressed_bytes)))
            hs = [h0] + [sd2.sd2_load_blob(blob) for _ in range(R - 1)]
            Wd0 = torch.from_numpy(np.where(mask != 0, W, np.uint16(0)).view(np.int16)).cuda().view(torch.bfloat16)
            Rd = max(2, int(np.ceil(4.0 * l2 / (2 * M * K))))
            Wd = [Wd0] + [Wd0.clone() for _ in range(Rd - 1)]
            for N in ns:
                X = torch.from_numpy(synth.make_activations(5, 0, 0, N, K).view(np.int16).copy()).cuda().view(torch.bfloat16)
                Y = torch.zeros((N, M), dtype=torch.bfloat16, device="cuda")

                def sparse_all():
                    for h in hs:
                        sd2.sd2_spmm(h, X, Y)

                def dense_all():
                    for w in Wd:
                        torch.matmul(X, w.t(), out=Y)

                us_s = time_graph(torch, sparse_all, 20) / R
                us_d = time_graph(torch, dense_all, 20) / Rd
                cross[N].append((sp, us_s, us_d))
                print("| %dx%d | %d | %.2f | %.3f | %.2f | %.0f | %.2f | %.2f |" % (
                    M, K, N, sp, h0.compressed_bytes / max(h0.nnz, 1), us_s, h0.compressed_bytes / us_s / 1e3, us_d, us_d / us_s), flush=True)
            for h in hs:
                sd2.sd2_free(h)
            del Wd, Wd0
            torch.cuda.empty_cache()
        for N in ns:
            pts = cross[N]
            where = "never on this grid"
            if pts[0][1] < pts[0][2]:
                where = "<= %.2f (already faster at the lowest grid point)" % pts[0][0]
            else:
                for (s0, a0, d0), (s1, a1, d1) in zip(pts, pts[1:]):
                    if a0 >= d0 and a1 < d1:
                        f0, f1 = a0 - d0, a1 - d1
                        where = "%.3f" % (s0 + (s1 - s0) * f0 / (f0 - f1))
                        break
            print("crossover %dx%d N=%d: sparse faster than cuBLAS dense from sparsity %s" % (M, K, N, where), flush=True)


if __name__ == "__main__":
    main()
