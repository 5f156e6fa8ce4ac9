"""Helpers shared by the GPU parity tests: moving seeded workloads to the device."""
import numpy as np
import torch

from paper_2608_18484_b200 import workloads as W


def heads_to_device(wl, heads, seed=0):
    """Returns (host list of (Q,K,V) float32 arrays, device tensors [1,H,N,d] in the workload dtype)."""
    host = [W.make_head(wl, h, seed) for h in heads]
    dt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    dev = []
    for t in range(3):
        x = torch.from_numpy(np.stack([hd[t] for hd in host])[None]).to(dt).cuda().contiguous()
        dev.append(x)
    return host, dev


def to_np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)
