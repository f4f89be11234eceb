"""An fp64 PyTorch restatement of the three synthetic SuperNets, used only to pin the C checker.

It is written against library routines (``torch.nn.functional.conv2d`` and friends) on tensors
that are first cut out of the blob with ordinary Python slices, so a wiring or indexing mistake in
the C code does not repeat here by construction.
"""
import numpy as np
import torch
import torch.nn.functional as F

from paper_2306_17266_b200 import workload as wl


def parse_blob(family, blob):
    words = np.frombuffer(np.ascontiguousarray(blob), dtype=np.uint32)
    recs = wl.supernet_records(family)
    pos = 8
    out = {}
    for r in recs:
        pos += 8
        f = words[pos:pos + r.n_floats].view(np.float32)
        d = {"w": torch.tensor(f[:r.n_weights].reshape(r.K, r.C, r.R, r.S), dtype=torch.float64)}
        q = r.n_weights
        if r.has_bn:
            for name in ("gamma", "beta", "mean", "var"):
                d[name] = torch.tensor(f[q:q + r.K], dtype=torch.float64)
                q += r.K
        if r.has_bias:
            d["bias"] = torch.tensor(f[q:q + r.K], dtype=torch.float64)
        out[r.name] = d
        pos += r.n_floats
    return out


def rnd8(x):
    return max(8, 8 * int(np.floor(x / 8 + 0.5)))


def hswish(x):
    return x * torch.clamp(x + 3, 0, 6) / 6


def bf16_store(x):
    """Round an fp64 tensor the way a bf16 store does: to fp32 first (the arithmetic type of the method), then
    to the nearest value with an 8-bit significand, ties to the even one.  Written out on the bit pattern."""
    bits = x.to(torch.float32).contiguous().view(torch.int32).to(torch.int64) & 0xFFFFFFFF
    bits = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000
    bits = torch.where(bits >= 2**31, bits - 2**32, bits).to(torch.int32)
    return bits.view(torch.float32).to(torch.float64)


# The tensors the bf16 mode STORES, and therefore rounds: every layer output after its epilogue ("layer"), the
# max-pooled map ("maxpool") and the SE-scaled map ("se_scale").  Pooled vectors, SE vectors, the head's mixing
# vector and the logits stay unrounded.  `skip` names points to leave out, so that a test can show what a
# forgotten rounding point does.
#
# `teacher` (name of a stored layer -> the tensor another implementation stored there, NHWC) turns the run into a
# layer-by-layer comparison: at every stored tensor the teacher has, the difference is recorded in `report` and the
# teacher's tensor is what the following layers consume.  Two correct implementations that add in different orders
# disagree on a few roundings per tensor, and in a deep network those few grow into differences as large as the
# rounding noise itself; fed with the same inputs, every single layer can be held to "a few one-step flips".
class Store:
    def __init__(self, on=False, skip=(), teacher=None):
        self.on, self.skip, self.teacher = on, set(skip), teacher
        self.report = {}

    def __call__(self, point, x, name=None):
        y = bf16_store(x) if self.on and point not in self.skip else x
        if self.teacher is not None and name in self.teacher:
            t = torch.tensor(np.asarray(self.teacher[name]), dtype=torch.float64).permute(0, 3, 1, 2)
            assert t.shape == y.shape, (name, t.shape, y.shape)
            diff = (t - y).abs()
            # one bf16 step at that magnitude; next to zero (an activation's kink) the fp32 noise of the sum itself
            step = torch.clamp(torch.maximum(t.abs(), y.abs()) * 2.0 ** -7, min=1e-5 * float(t.abs().max()))
            self.report[name] = {"n": t.numel(), "unequal": int((diff > 0).sum()), "beyond_one_step": int((diff > step).sum()),
                                 "max_abs": float(diff.max())}
            return t
        return y


NO_STORE = Store(False)


def conv(P, name, x, Kp, k, stride, act=None, res=None, groups=1, store=NO_STORE):
    """x NCHW. Slice K' filters, matching input channels, centre k x k window; conv; BN; +res; act."""
    d = P[name]
    R = d["w"].shape[2]
    o = (R - k) // 2
    Cp = 1 if groups > 1 else x.shape[1]
    w = d["w"][:Kp, :Cp, o:o + k, o:o + k]
    y = F.conv2d(x, w, stride=stride, padding=(k - 1) // 2, groups=groups)
    if "gamma" in d:
        y = F.batch_norm(y, d["mean"][:Kp].clone(), d["var"][:Kp].clone(), d["gamma"][:Kp], d["beta"][:Kp], False, 0.0, 1e-5)
    if "bias" in d:
        y = y + d["bias"][:Kp].view(1, -1, 1, 1)
    if res is not None:
        y = y + res
    if act == "relu":
        y = F.relu(y)
    elif act == "hswish":
        y = hswish(y)
    return store("layer", y, name)


def linear(P, name, v, Kp):
    d = P[name]
    return v @ d["w"][:Kp, :v.shape[1], 0, 0].T + d["bias"][:Kp]


def forward(family, P, cfg, x_nhwc, store=NO_STORE):
    x = torch.tensor(np.asarray(x_nhwc), dtype=torch.float64).permute(0, 3, 1, 2)
    if family == wl.TINY:
        w = [int(wl.TINY_WIDTHS[s] * float(cfg.width[s + 1])) for s in range(3)]
        x = conv(P, "stem", x, w[0], 3, 1, "relu", store=store)
        for s in range(3):
            for b in range(cfg.depth[s]):
                st = 2 if (b == 0 and s > 0) else 1
                sc = conv(P, f"s{s}b{b}.proj", x, w[s], 1, st, store=store) if (b == 0 and s > 0) else x
                t = conv(P, f"s{s}b{b}.conv1", x, w[s], 3, st, "relu", store=store)
                x = conv(P, f"s{s}b{b}.conv2", t, w[s], 3, 1, "relu", res=sc, store=store)
        return linear(P, "fc", x.mean(dim=(2, 3)), 10).numpy()
    if family == wl.RESNET:
        x = conv(P, "stem", x, rnd8(64 * float(cfg.width[0])), 7, 2, "relu", store=store)
        x = store("maxpool", F.max_pool2d(x, 3, 2, 1))
        for s in range(4):
            out = rnd8(wl.RESNET_BASE[s] * float(cfg.width[s + 1]))
            for b in range(cfg.depth[s]):
                st = 2 if (b == 0 and s > 0) else 1
                mid = rnd8(out * float(cfg.expand[s][b]))
                sc = conv(P, f"s{s}b{b}.proj", x, out, 1, st, store=store) if b == 0 else x
                t = conv(P, f"s{s}b{b}.conv1", x, mid, 1, 1, "relu", store=store)
                t = conv(P, f"s{s}b{b}.conv2", t, mid, 3, st, "relu", store=store)
                x = conv(P, f"s{s}b{b}.conv3", t, out, 1, 1, "relu", res=sc, store=store)
        return linear(P, "fc", x.mean(dim=(2, 3)), 1000).numpy()
    acts = ["relu", "relu", "hswish", "hswish", "hswish"]
    strides = [2, 2, 2, 1, 2]
    x = conv(P, "stem", x, 16, 3, 2, "hswish", store=store)
    t = conv(P, "first.dw", x, 16, 3, 1, "relu", groups=16, store=store)
    x = conv(P, "first.pw", t, 16, 1, 1, None, res=x, store=store)
    for s in range(5):
        out = wl.MBV3_OUT[s]
        for b in range(cfg.depth[s]):
            st = strides[s] if b == 0 else 1
            cin = x.shape[1]
            mid = rnd8(cin * float(cfg.expand[s][b]))
            t = conv(P, f"s{s}b{b}.expand", x, mid, 1, 1, acts[s], store=store)
            t = conv(P, f"s{s}b{b}.dw", t, mid, int(cfg.kernel[s][b]), st, acts[s], groups=mid, store=store)
            if wl.MBV3_SE[s]:
                sq = rnd8(mid / 4)
                g = t.mean(dim=(2, 3))
                g = F.relu(linear(P, f"s{s}b{b}.se1", g, sq))
                g = torch.clamp(linear(P, f"s{s}b{b}.se2", g, mid) + 3, 0, 6) / 6
                t = store("se_scale", t * g.view(g.shape[0], -1, 1, 1), f"s{s}b{b}.se2")
            x = conv(P, f"s{s}b{b}.project", t, out, 1, 1, None, res=x if (st == 1 and cin == out) else None, store=store)
    t = conv(P, "head.conv", x, 960, 1, 1, "hswish", store=store)
    v = hswish(linear(P, "head.mix", t.mean(dim=(2, 3)), 1280))
    return linear(P, "fc", v, 1000).numpy()
