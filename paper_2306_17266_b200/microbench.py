"""Per-layer timing of the sliced convolution and depthwise kernels through sgs_conv2d_sliced.

    python -m paper_2306_17266_b200.microbench conv --preset resnet_b1
    python -m paper_2306_17266_b200.microbench conv --shape 1,7,7,720,720,720,720,3,3,1 --once 3
    python -m paper_2306_17266_b200.microbench conv-i8 --preset resnet_b16
    python -m paper_2306_17266_b200.microbench dw --preset large

conv shapes: N,H,W,Cmax,C,Kmax,K,R,k,stride; dw shapes: N,H,W,K,k,stride (stored kernel 7x7).
Times are CUDA events around a captured graph of back-to-back launches (conv) or a plain launch loop
(dw, working sets larger than L2).  `--once n` just runs n launches (for profilers).
"""
from __future__ import annotations

import argparse

import torch

from . import binding as sgs

CONV_PRESETS = {
    # layer shapes of the ResNet-50-shaped SuperNet at batch 1 (mean-ish SubNet widths)
    "resnet_b1": [(1, 56, 56, 64, 64, 88, 64, 1, 1, 1), (1, 56, 56, 88, 88, 88, 88, 3, 3, 1), (1, 56, 56, 88, 88, 256, 208, 1, 1, 1),
                  (1, 28, 28, 176, 176, 176, 176, 3, 3, 1), (1, 14, 14, 360, 360, 360, 360, 3, 3, 1), (1, 14, 14, 1024, 1024, 360, 360, 1, 1, 1),
                  (1, 7, 7, 720, 720, 720, 720, 3, 3, 1), (1, 7, 7, 720, 720, 2048, 2048, 1, 1, 1), (1, 14, 14, 1024, 816, 2048, 1640, 1, 1, 2)],
    # the same layers at batch 16 and 64
    "resnet_b16": [(16, 56, 56, 88, 88, 88, 88, 3, 3, 1), (16, 14, 14, 360, 360, 1024, 1024, 1, 1, 1), (16, 28, 28, 176, 176, 176, 176, 3, 3, 1)],
    "resnet_b64": [(64, 28, 28, 176, 176, 176, 176, 3, 3, 1), (64, 56, 56, 64, 64, 256, 256, 1, 1, 1), (64, 14, 14, 360, 360, 360, 360, 3, 3, 1)],
}
DW_PRESETS = {
    "large": [(64, 56, 56, 480, k, s) for k in (3, 5, 7) for s in (1, 2)] + [(128, 28, 28, 672, k, 1) for k in (3, 5, 7)],
    "b1": [(1, 112, 112, 96, 3, 2), (1, 28, 28, 240, 5, 1), (1, 14, 14, 672, 7, 1)],
}


def _conv_tensors(shape):
    N, H, W, Cmax, C, Kmax, K, R, k, stride = shape
    p = (k - 1) // 2
    Ho, Wo = (H + 2 * p - k) // stride + 1, (W + 2 * p - k) // stride + 1
    x = torch.randn(N, H, W, C, device="cuda").to(torch.bfloat16)
    w = (torch.randn(Kmax, R, R, Cmax, device="cuda") * 0.05).to(torch.bfloat16)
    sc, sh = torch.ones(Kmax, device="cuda"), torch.zeros(Kmax, device="cuda")
    y = torch.empty(N, Ho, Wo, K, device="cuda", dtype=torch.bfloat16)
    return x, w, sc, sh, y, Ho, Wo


def bench_conv(shape, iters=200, once=0, split_off=0, impl=2):
    N, H, W, Cmax, C, Kmax, K, R, k, stride = shape
    x, w, sc, sh, y, Ho, Wo = _conv_tensors(shape)
    d = sgs.ConvDesc(N=N, H=H, W=W, C=C, K=K, Kmax=Kmax, Cmax=Cmax, R=R, k=k, stride=stride, act=1, dtype=sgs.SGS_BF16, impl=impl,
                     depthwise=0, cache_k=0, cache_c=0, weight_policy=0, split_k_off=split_off)
    st = torch.cuda.Stream()

    def launch(stream):
        sgs.conv2d_sliced(d, x.data_ptr(), w.data_ptr(), sc.data_ptr(), sh.data_ptr(), 0, y.data_ptr(), stream)

    with torch.cuda.stream(st):
        for _ in range(max(once, 3)):
            launch(st.cuda_stream)
    torch.cuda.synchronize()
    if once:
        return None
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        for _ in range(iters):
            launch(st.cuda_stream)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    g.replay()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1000 / iters
    flops = 2.0 * N * Ho * Wo * K * C * k * k
    nbytes = 2.0 * (N * H * W * C + N * Ho * Wo * K + K * C * k * k)
    return {"shape": shape, "us": us, "tflops": flops / us / 1e6, "gbs": nbytes / us / 1e3}


def bench_conv_i8(shape, iters=200):
    """The same layer shapes with 8-bit operands (sgs_conv2d_sliced_i8); channel counts are rounded up to 16."""
    N, H, W, Cmax, C, Kmax, K, R, k, stride = shape
    r16 = lambda v: (v + 15) // 16 * 16
    Cmax, C = r16(Cmax), r16(C)
    p = (k - 1) // 2
    Ho, Wo = (H + 2 * p - k) // stride + 1, (W + 2 * p - k) // stride + 1
    x = torch.randint(0, 256, (N, H, W, C), device="cuda", dtype=torch.uint8)
    w = torch.randint(-127, 128, (Kmax, R, R, Cmax), device="cuda", dtype=torch.int8)
    mult = torch.full((Kmax,), 1 << 30, device="cuda", dtype=torch.int32)
    shift = torch.full((Kmax,), 12, device="cuda", dtype=torch.int32)
    bias = torch.zeros(Kmax, device="cuda", dtype=torch.int32)
    y = torch.empty(N, Ho, Wo, K, device="cuda", dtype=torch.uint8)
    d = sgs.ConvI8Desc(N=N, H=H, W=W, C=C, K=K, Kmax=Kmax, Cmax=Cmax, R=R, k=k, stride=stride, relu=1)
    st = torch.cuda.Stream()

    def launch(stream):
        sgs.conv2d_sliced_i8(d, x.data_ptr(), w.data_ptr(), mult.data_ptr(), shift.data_ptr(), bias.data_ptr(), 0, y.data_ptr(), stream)

    with torch.cuda.stream(st):
        for _ in range(3):
            launch(st.cuda_stream)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        for _ in range(iters):
            launch(st.cuda_stream)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    g.replay()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1000 / iters
    ops = 2.0 * N * Ho * Wo * K * C * k * k
    nbytes = 1.0 * (N * H * W * C + N * Ho * Wo * K + K * C * k * k)
    return {"shape": (N, H, W, Cmax, C, Kmax, K, R, k, stride), "us": us, "tops": ops / us / 1e6, "gbs": nbytes / us / 1e3}


def bench_dw(shape, iters=20, once=0):
    N, H, W, K, k, stride = shape
    p = (k - 1) // 2
    Ho, Wo = (H + 2 * p - k) // stride + 1, (W + 2 * p - k) // stride + 1
    x = torch.randn(N, H, W, K, device="cuda").to(torch.bfloat16)
    w = (torch.randn(7, 7, K, device="cuda") * 0.1).to(torch.bfloat16)
    sc, sh = torch.ones(K, device="cuda"), torch.zeros(K, device="cuda")
    y = torch.empty(N, Ho, Wo, K, device="cuda", dtype=torch.bfloat16)
    d = sgs.ConvDesc(N=N, H=H, W=W, C=1, K=K, Kmax=K, Cmax=1, R=7, k=k, stride=stride, act=2, dtype=sgs.SGS_BF16, impl=0, depthwise=1,
                     cache_k=0, cache_c=0, weight_policy=0, split_k_off=0)
    s = torch.cuda.current_stream().cuda_stream
    for _ in range(max(once, 3)):
        sgs.conv2d_sliced(d, x.data_ptr(), w.data_ptr(), sc.data_ptr(), sh.data_ptr(), 0, y.data_ptr(), s)
    torch.cuda.synchronize()
    if once:
        return None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        sgs.conv2d_sliced(d, x.data_ptr(), w.data_ptr(), sc.data_ptr(), sh.data_ptr(), 0, y.data_ptr(), s)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1000 / iters
    nbytes = 2.0 * (x.numel() + y.numel())
    return {"shape": shape, "us": us, "gbs": nbytes / us / 1e3, "mbytes": nbytes / 1e6}


def wave_trace(family, wave, queries, res, batch):
    """Per-layer device time of a stream run as waves (one wave at a time, every launch between two events)."""
    from . import workload as wl
    fam = {"resnet": wl.RESNET, "mbv3": wl.MBV3}[family]
    net = sgs.SuperNet(fam, wl.make_blob(fam, seed=0, bf16_weights=True), sgs.SGS_BF16)
    cfgs = wl.cfg_array(wl.uniform_stream(fam, queries, seed=2 if fam == wl.RESNET else 3))
    x = torch.from_numpy(wl.make_inputs(queries, batch, res, seed=1, bf16=True).reshape(queries * batch, res, res, 3)).cuda().to(torch.bfloat16).contiguous()
    out = torch.zeros((queries * batch, 1000), dtype=torch.float32, device="cuda")
    st = torch.cuda.Stream()
    opts = sgs.StreamOpts(cache_enabled=1, window_q=4, record_latency=0, concurrency=1, wave=wave)
    for _ in range(2):
        net.stream_run(cfgs, x.data_ptr(), batch, res, out.data_ptr(), opts, st.cuda_stream)
    net.set_option("profile", 2)
    net.stream_run(cfgs, x.data_ptr(), batch, res, out.data_ptr(), opts, st.cuda_stream)
    recs = net.profile_trace()
    net.set_option("profile", 0)
    rows, order = {}, []
    for r in recs:
        key = (r["kernel_class"], r["name"] or "(no weights)")
        if key not in rows:
            rows[key] = {"n": 0, "ms": 0.0, "bytes": 0.0, "flops": 0.0, "members": 0, "tiles": 0}
            order.append(key)
        a = rows[key]
        a["n"] += 1; a["ms"] += r["ms"]; a["bytes"] += r["alg_bytes"]; a["flops"] += r["flops"]; a["members"] += r["members"]; a["tiles"] += r["tiles"]
    total = sum(a["ms"] for a in rows.values())
    names = ["conv_tc", "conv_cuda_core", "depthwise", "other"]
    print(f"{family}: {queries} queries, waves of {wave}, batch {batch}, {res}x{res}: {len(recs)} launches, {total:.2f} ms of kernel time")
    for key in order:
        a = rows[key]
        print(f"{names[key[0]]:10s} {key[1]:28s} launches {a['n']:4d}  members {a['members'] / a['n']:5.1f}  tiles {a['tiles'] / a['n']:7.1f}  "
              f"{1e3 * a['ms'] / a['n']:7.1f} us  {100 * a['ms'] / total:5.1f} %  {a['bytes'] / a['ms'] / 1e6:8.1f} GB/s  {a['flops'] / a['ms'] / 1e9:7.1f} TFLOP/s")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kind", choices=["conv", "conv-i8", "dw", "trace"])
    ap.add_argument("--family", default="resnet", choices=["resnet", "mbv3"])
    ap.add_argument("--wave", type=int, default=32)
    ap.add_argument("--queries", type=int, default=128)
    ap.add_argument("--res", type=int, default=224)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--preset", default=None)
    ap.add_argument("--shape", default=None, help="comma-separated shape")
    ap.add_argument("--once", type=int, default=0, help="only run this many launches (profiling)")
    ap.add_argument("--split-off", type=int, default=0)
    args = ap.parse_args()
    if args.kind == "trace":
        wave_trace(args.family, args.wave, args.queries, args.res, args.batch)
        return
    if args.shape:
        shapes = [tuple(int(v) for v in args.shape.split(","))]
    else:
        table = DW_PRESETS if args.kind == "dw" else CONV_PRESETS
        shapes = table[args.preset or ("large" if args.kind == "dw" else "resnet_b1")]
    for sh in shapes:
        if args.kind == "conv-i8":
            r = bench_conv_i8(sh)
            sh = r["shape"]
            print(f"conv-i8 N{sh[0]} {sh[1]}x{sh[2]} C{sh[4]} K{sh[6]} k{sh[8]} s{sh[9]}: {r['us']:8.2f} us  {r['tops']:8.2f} TOP/s  {r['gbs']:8.1f} GB/s", flush=True)
        elif args.kind == "conv":
            r = bench_conv(sh, once=args.once, split_off=args.split_off)
            if r:
                print(f"conv N{sh[0]} {sh[1]}x{sh[2]} C{sh[4]} K{sh[6]} k{sh[8]} s{sh[9]}: {r['us']:8.2f} us  {r['tflops']:8.2f} TFLOP/s  {r['gbs']:8.1f} GB/s", flush=True)
        else:
            r = bench_dw(sh, once=args.once)
            if r:
                print(f"dw N{sh[0]} {sh[1]}x{sh[2]} C{sh[3]} k{sh[4]} s{sh[5]}: {r['us']:8.1f} us  {r['gbs']:8.1f} GB/s  ({r['mbytes']:.0f} MB)", flush=True)
    if args.once:
        print("ok")


if __name__ == "__main__":
    main()
