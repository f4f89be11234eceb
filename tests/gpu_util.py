"""Helpers of the GPU parity tests: device buffers through torch, parity metrics."""
import numpy as np
import torch

import oracle
import paper_2306_17266_b200 as sgs
from paper_2306_17266_b200 import workload as wl

_cache = {}


def nets(family, bf16, seed=0):
    """(blob, oracle net, GPU net) for a family; cached per test session."""
    key = (family, bf16, seed)
    if key not in _cache:
        blob = wl.make_blob(family, seed=seed, bf16_weights=bf16)
        _cache[key] = (blob, oracle.Net(family, blob), sgs.SuperNet(family, blob, sgs.SGS_BF16 if bf16 else sgs.SGS_F32))
    return _cache[key]


def to_device(x_np, bf16):
    t = torch.from_numpy(np.ascontiguousarray(x_np)).cuda()
    return t.to(torch.bfloat16).contiguous() if bf16 else t.contiguous()


def gpu_forward(gnet, cfg, x_np, bf16):
    """x_np: (batch, res, res, 3) float32 -> logits (batch, classes) float32 via sgs_subnet_run."""
    x = to_device(x_np, bf16)
    out = torch.empty((x.shape[0], gnet.n_classes), dtype=torch.float32, device="cuda")
    gnet.subnet_run(cfg, x.data_ptr(), x.shape[0], x.shape[1], out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def rel_err(got, ref):
    """max |err| / max |ref| per output row, worst row."""
    return float(np.max(np.abs(got - ref).max(axis=-1) / np.maximum(np.abs(ref).max(axis=-1), 1e-30)))


def argmax_agreement(got, ref):
    return float(np.mean(got.argmax(-1) == ref.argmax(-1)))
