"""Helpers shared by the GPU parity tests: moving seeded workloads to the device."""
import numpy as np
import torch

from paper_2608_18484_b200 import workloads as W


def heads_to_device(wl, heads, seed=0, step=0):
    """Returns (host list of (Q,K,V) float32 arrays, device tensors [1,H,N,d] in the workload dtype)."""
    host = [W.make_head(wl, h, seed, step) for h in heads]
    dt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    dev = []
    for t in range(3):
        x = torch.from_numpy(np.stack([hd[t] for hd in host])[None]).to(dt).cuda().contiguous()
        dev.append(x)
    return host, dev


def to_np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def assert_bf16_close(O, ref):
    """bf16 tensors, float32 accumulation, bf16 output: relative L2 <= 1e-2 and, element by element,
    |O - ref| <= 2e-2 -- except where the reference element is so large that a single correctly rounded
    bf16 store already exceeds that (half an ulp is 2^-9 |o| rounded up to a power of two: 0.031 for
    8 <= |o| < 16); there the bound is one bf16 ulp, 2^-7 |ref|."""
    from oracle import sparsepr_oracle as orc
    err = orc.rel_l2(O, ref)
    assert err <= 1e-2, err
    excess = np.abs(O - ref) - np.maximum(2e-2, 2.0 ** -7 * np.abs(ref))
    assert excess.max() <= 0.0, (float(np.abs(O - ref).max()), float(excess.max()))
