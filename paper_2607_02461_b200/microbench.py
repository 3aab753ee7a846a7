"""Per-kernel micro-benchmarks (device-timed with CUDA events, L2 flushed between iterations).

    python -m paper_2607_02461_b200.microbench rq   --tokens 17776 --dim 3072 --bits 4 --block 128
    python -m paper_2607_02461_b200.microbench gemm --tokens 4608 --dim 3072 --m 9216 --bits-a 4 --bits-w 4
    python -m paper_2607_02461_b200.microbench sweep [--quick]     # rotate+quantize bandwidth sweep
    python -m paper_2607_02461_b200.microbench adaln --tokens 1 --dim 3072 --m 18432   # AdaLN INT4 projection
    python -m paper_2607_02461_b200.microbench step --shape wan --bits-a 6             # whole block step, W4A6 or W4A4
    python -m paper_2607_02461_b200.microbench ks --tokens 512 --dim 3072              # KS distance of rotated coordinates to f_d

Inputs are synthetic and generated on the GPU (normal values, per-token log-uniform scale, 1% of the
channels multiplied by 30); these runs time the kernels, parity is covered by the tests.
Each run prints one JSON line per point.
"""
import argparse
import json
import sys

import torch

from . import binding as B
from . import build as oqbuild


def gen_x(n, d, seed=0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    x = torch.randn((n, d), device="cuda", generator=g)
    x *= torch.exp(torch.empty(n, 1, device="cuda").uniform_(-2.3026, 2.3026, generator=g))
    ch = torch.randperm(d, device="cuda", generator=g)[: max(1, d // 100)]
    x[:, ch] *= 30.0
    return x.to(torch.bfloat16)


def time_kernel(fn, iters, warmup=3, flush_mb=256):
    flush = torch.empty(flush_mb << 20, dtype=torch.uint8, device="cuda")
    for _ in range(warmup):
        fn()
    ts = []
    for _ in range(iters):
        flush.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); fn(); b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    ts.sort()
    return ts[len(ts) // 2], ts[0]


def run_rq(n, d, bits, block, iters):
    rot, cb = B.oq_make_rpbh(d, block, 0), B.oq_build_codebook(d, bits)
    X = gen_x(n, d)
    nrm = torch.empty(n, dtype=torch.float32, device="cuda")
    if bits == 6:      # 64 levels: the output is the bf16 level matrix
        lev = torch.empty((n, d), dtype=torch.bfloat16, device="cuda")
        med, best = time_kernel(lambda: B.oq_rotate_quantize_act_levels(X, rot, cb, out=lev, out_norm=nrm), iters)
        nbytes = 2 * n * d + 2 * n * d + 4 * n
    else:
        idx = torch.empty((n, B.oq_packed_bytes(n, d, bits)[1]), dtype=torch.uint8, device="cuda")
        med, best = time_kernel(lambda: B.oq_rotate_quantize_act(X, rot, cb, out_idx=idx, out_norm=nrm), iters)
        nbytes = 2 * n * d + n * d * bits // 8 + 4 * n
    return {"kernel": "rotate_quantize", "tokens": n, "dim": d, "bits": bits, "block": block, "ms_median": med,
            "ms_min": best, "bytes": nbytes, "gbs": nbytes / med / 1e6, "gbs_best": nbytes / best / 1e6}


def run_gemm(n, d, m, ba, bw, iters, levels=False):
    rot = B.oq_make_rpbh(d, 128, 0)
    cba, cbw = B.oq_build_codebook(d, ba), B.oq_build_codebook(d, bw)
    xq, xs = B.oq_rotate_quantize_act(gen_x(n, d), rot, cba)
    W = (torch.randn((m, d), device="cuda") * 0.02).to(torch.bfloat16)
    wq, wr = B.oq_quantize_weights(W, rot, cbw)
    del W
    Y = torch.empty((n, m), dtype=torch.bfloat16, device="cuda")
    if levels:
        xd = B.oq_decode_levels(xq, n, d, cba)
        med, best = time_kernel(lambda: B.oq_qlinear_levels(xd, xs, wq, wr, cbw, d, out=Y), iters)
    else:
        med, best = time_kernel(lambda: B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d, out=Y), iters)
    fl = 2.0 * n * m * d
    return {"kernel": "qlinear_levels" if levels else "qlinear", "tokens": n, "dim": d, "m": m, "bits_a": ba, "bits_w": bw, "ms_median": med,
            "ms_min": best, "flops": fl, "tflops": fl / med / 1e9, "tflops_best": fl / best / 1e9}


def run_adaln(n, d, m, iters):
    W = (torch.randn((m, d), device="cuda") * 0.02).to(torch.bfloat16)
    Wq, Sc = B.oq_adaln_quantize_weights(W)
    del W
    X = torch.nn.functional.silu(torch.randn((n, d), device="cuda")).to(torch.bfloat16)
    Y = torch.empty((n, m), dtype=torch.bfloat16, device="cuda")
    med, best = time_kernel(lambda: B.oq_adaln_linear(X, Wq, Sc, m, out=Y), iters)
    passes = (n + 7) // 8
    nbytes = passes * (m * d // 2 + 2 * m * d // 64) + 2 * n * d + 2 * n * m
    return {"kernel": "adaln_linear", "tokens": n, "dim": d, "m": m, "ms_median": med, "ms_min": best, "bytes": nbytes,
            "gbs": nbytes / med / 1e6, "gbs_best": nbytes / best / 1e6}


def run_step(shape, ba, bw, iters, split_qkv=False):
    """The linears of one FLUX- or Wan-shaped block through oq_block_forward (one stream, every input rotated and
    quantized once).  6-bit activations travel as bf16 levels, 2-4-bit ones packed.  split_qkv: the fused qkv layer
    becomes three projections that share one quantized input."""
    from . import synth
    tokens, layers = (synth.FLUX_TOKENS, synth.FLUX_LAYERS) if shape == "flux" else (synth.WAN_TOKENS, synth.WAN_LAYERS)
    inputs, lys = [], []
    for name, d, m in layers:
        rot = B.oq_make_rpbh(d, 128, 0)
        cba, cbw = B.oq_build_codebook(d, ba), B.oq_build_codebook(d, bw)
        xq = (torch.empty((tokens, d), dtype=torch.bfloat16, device="cuda") if ba == 6
              else torch.empty((tokens, B.oq_packed_bytes(tokens, d, ba)[1]), dtype=torch.uint8, device="cuda"))
        inputs.append(dict(X=gen_x(tokens, d), rot=rot, cb_a=cba, xq=xq, xs=torch.empty(tokens, dtype=torch.float32, device="cuda")))
        for mm in ([m // 3] * 3 if (split_qkv and name == "qkv") else [m]):
            W = (torch.randn((mm, d), device="cuda") * 0.02).to(torch.bfloat16)
            wq, wr = B.oq_quantize_weights(W, rot, cbw)
            del W
            lys.append(dict(input=len(inputs) - 1, wq=wq, wr=wr, cb_w=cbw, d=d, m=mm,
                            Y=torch.empty((tokens, mm), dtype=torch.bfloat16, device="cuda")))
    med, best = time_kernel(lambda: B.oq_block_forward(inputs, lys), iters)
    fl = sum(2.0 * tokens * l["m"] * l["d"] for l in lys)
    return {"kernel": "block_step", "shape": shape, "tokens": tokens, "bits_a": ba, "bits_w": bw, "layers": len(lys),
            "inputs": len(inputs), "ms_median": med, "ms_min": best, "flops": fl, "tflops": fl / med / 1e9,
            "tflops_best": fl / best / 1e9}


def run_ks(n, d, blocks):
    """Diagnostic in the spirit of the paper's KS-distance figure: how close the coordinates of the rotated, normalised
    tokens come to the marginal f_d that the codebook was fitted to (Eq. 2), per block size and with / without the
    synthetic channel outliers.  Kolmogorov-Smirnov distance of each token's d coordinates to the cdf
    F_d(t) = 1/2 + sgn(t) I_{t^2}(1/2, (d-1)/2) / 2, summarised over the tokens.  Uses the rotated values that
    oq_rotate_quantize_act exports for the tests."""
    import numpy as np
    from scipy.special import betainc
    out = []
    g = torch.Generator(device="cuda").manual_seed(1)
    plain = torch.randn((n, d), device="cuda", generator=g).to(torch.bfloat16)
    for name, X in (("outliers_x30", gen_x(n, d)), ("gaussian", plain)):
        for block in blocks:
            if d % block:
                continue
            rot, cb = B.oq_make_rpbh(d, block, 0), B.oq_build_codebook(d, 4)
            z = torch.empty((n, d), dtype=torch.float32, device="cuda")
            _, s = B.oq_rotate_quantize_act(X, rot, cb, dbg_rotated=z)
            t = np.sort((z / (s[:, None] + 1e-10)).double().cpu().numpy(), axis=1)
            cdf = 0.5 + 0.5 * np.sign(t) * betainc(0.5, (d - 1) / 2.0, t * t)
            i = np.arange(1, d + 1)[None, :] / d
            ks = np.maximum(np.abs(cdf - i), np.abs(cdf - (i - 1.0 / d))).max(axis=1)
            out.append({"kernel": "ks_distance", "input": name, "tokens": n, "dim": d, "block": block,
                        "ks_median": float(np.median(ks)), "ks_max": float(ks.max()),
                        "ks_of_a_perfect_sample": float(0.87 / np.sqrt(d))})
    return out


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("mode", choices=["rq", "gemm", "sweep", "adaln", "step", "ks"])
    ap.add_argument("--tokens", type=int, default=17776)
    ap.add_argument("--dim", type=int, default=3072)
    ap.add_argument("--m", type=int, default=9216)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--bits-a", type=int, default=4)
    ap.add_argument("--bits-w", type=int, default=4)
    ap.add_argument("--block", type=int, default=128)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--shape", choices=["flux", "wan"], default="wan")
    ap.add_argument("--levels", action="store_true", help="gemm: activations as bf16 levels (oq_qlinear_levels)")
    ap.add_argument("--split-qkv", action="store_true", help="step: q, k, v as three layers that share one quantized input")
    ap.add_argument("--kernel", type=int, default=0, help="rotate+quantize kernel: 0 auto, 1 general, 2 registers, 3 tensor cores")
    a = ap.parse_args(argv)
    oqbuild.build()
    B.oq_debug_select_rq_kernel(a.kernel)
    if a.mode == "rq":
        print(json.dumps(run_rq(a.tokens, a.dim, a.bits, a.block, a.iters)))
    elif a.mode == "gemm":
        print(json.dumps(run_gemm(a.tokens, a.dim, a.m, a.bits_a, a.bits_w, a.iters, a.levels)))
    elif a.mode == "step":
        print(json.dumps(run_step(a.shape, a.bits_a, a.bits_w, a.iters, a.split_qkv)))
    elif a.mode == "ks":
        for r in run_ks(a.tokens, a.dim, [64, 128, 256, 1024]):
            print(json.dumps(r))
    elif a.mode == "adaln":
        print(json.dumps(run_adaln(a.tokens, a.dim, a.m, a.iters)))
    else:
        toks = [4608, 32760] if a.quick else [4608, 17776, 32760, 75600]
        for n in toks:
            for d in [1024, 3072, 5120, 12288, 13824]:
                for bits in [3, 4]:
                    for block in [64, 128, 256]:
                        print(json.dumps(run_rq(n, d, bits, block, a.iters)))
                        sys.stdout.flush()
                        torch.cuda.empty_cache()
    assert B.oq_device_status() == 0


if __name__ == "__main__":
    main()
