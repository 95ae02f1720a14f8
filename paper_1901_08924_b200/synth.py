"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random inputs; it contains none of the method's arithmetic and imports
neither the CUDA binding nor the CPU oracle, so both sides can be fed from it.

The paper's linear-model experiments (Section 5.1) use dense synthetic regression data with
i.i.d. noise, and its gradient histograms (Figure 2) are close to Gaussian; the generators here
reproduce those shapes and value distributions, not any dataset's records.

Every generator takes `device`: "cpu" gives numpy-backed torch CPU tensors; "cuda" draws on the
GPU with a seeded torch.Generator (values differ between devices for the same seed, so a test
draws once and copies).
"""
import math

import torch


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def linear_problem(n, d, loss="logistic", sparsity=0.1, noise=0.1, seed=0, col_scale_range=None,
                   device="cpu", chunk_rows=16384):
    """Dense X (n x d, fp32, i.i.d. N(0, 1/d)), planted sparse w*, labels from X w* + noise.

    loss "logistic": y = sign(X w* + noise * N(0,1)) in {-1,+1};  "least_squares": y = X w* + noise * N(0,1).
    col_scale_range=(lo, hi): multiply column j by a scale drawn log-uniformly in [lo, hi]
    (ill-conditioned design).
    Returns (X, y, w_star) as fp32 tensors on `device`.
    """
    g = _gen(seed, device)
    w = torch.randn(d, generator=g, device=device, dtype=torch.float32)
    keep = torch.rand(d, generator=g, device=device) < sparsity
    w = torch.where(keep, w, torch.zeros_like(w))
    scale = None
    if col_scale_range is not None:
        lo, hi = col_scale_range
        e = torch.rand(d, generator=g, device=device, dtype=torch.float32)
        scale = torch.exp(math.log(lo) + e * (math.log(hi) - math.log(lo)))
    X = torch.empty((n, d), device=device, dtype=torch.float32)
    y = torch.empty(n, device=device, dtype=torch.float32)
    inv_sqrt_d = 1.0 / math.sqrt(d)
    for r0 in range(0, n, chunk_rows):
        r1 = min(n, r0 + chunk_rows)
        blk = torch.randn((r1 - r0, d), generator=g, device=device, dtype=torch.float32) * inv_sqrt_d
        if scale is not None:
            blk = blk * scale
        X[r0:r1] = blk
        t = blk @ w + noise * torch.randn(r1 - r0, generator=g, device=device, dtype=torch.float32)
        y[r0:r1] = torch.where(t >= 0, torch.ones_like(t), -torch.ones_like(t)) if loss == "logistic" else t
    return X, y, w


def gradient_vectors(N, length, dist="gauss", seed=0, device="cpu"):
    """N worker gradient vectors of `length` fp32 values: N(0,1) or Student-t with 3 degrees of freedom."""
    g = _gen(seed, device)
    U = torch.randn((N, length), generator=g, device=device, dtype=torch.float32)
    if dist == "student_t3":
        for i in range(N):  # z / sqrt(chi2_3 / 3), one worker at a time to bound memory
            c = torch.zeros(length, device=device, dtype=torch.float32)
            for _ in range(3):
                c += torch.randn(length, generator=g, device=device, dtype=torch.float32) ** 2
            U[i] /= torch.sqrt(c / 3.0)
    elif dist != "gauss":
        raise ValueError(dist)
    return U


def resnet18_shapes(num_classes=1000):
    """The 62 parameter tensors of an 18-layer residual network with a `num_classes`-way head.

    Derived from the architecture: a 7x7 stem convolution (3->64) with its normalisation, four
    stages of two basic blocks (two 3x3 convolutions each, widths 64/128/256/512, each followed by
    a normalisation layer with a scale and a shift vector), a 1x1 projection convolution with
    normalisation on the first block of stages 2-4, and a fully connected head with bias.
    """
    shapes = [(64, 3, 7, 7), (64,), (64,)]
    width_in = 64
    for stage, width in enumerate((64, 128, 256, 512)):
        for block in range(2):
            cin = width_in if block == 0 else width
            shapes += [(width, cin, 3, 3), (width,), (width,), (width, width, 3, 3), (width,), (width,)]
            if block == 0 and stage > 0:
                shapes += [(width, cin, 1, 1), (width,), (width,)]
        width_in = width
    shapes += [(num_classes, 512), (num_classes,)]
    return shapes


def segment_offsets(shapes):
    offs = [0]
    for s in shapes:
        offs.append(offs[-1] + math.prod(s))
    return offs


def dnn_gradients(N, shapes=None, seed=0, device="cpu", sigma_range=(1e-4, 1e-1)):
    """Layer-wise gradient triples for the SVRG estimator on a DNN-shaped parameter list.

    Per tensor l a scale sigma_l is drawn log-uniformly in sigma_range; per worker i the current
    and the snapshot minibatch gradients are N(0, sigma_l) vectors; mu is the mean over workers of
    a third such vector (the snapshot full gradient).  Returns (cur, snap, mu, offsets): cur and
    snap are (N, total) fp32, mu is (total,), offsets has len(shapes)+1 entries.
    """
    shapes = resnet18_shapes() if shapes is None else shapes
    offs = segment_offsets(shapes)
    total = offs[-1]
    g = _gen(seed, device)
    e = torch.rand(len(shapes), generator=g, device=device, dtype=torch.float32)
    lo, hi = sigma_range
    sig = torch.exp(math.log(lo) + e * (math.log(hi) - math.log(lo)))
    lens = torch.tensor([offs[i + 1] - offs[i] for i in range(len(shapes))], device=device)
    sig_full = torch.repeat_interleave(sig, lens)
    cur = torch.randn((N, total), generator=g, device=device, dtype=torch.float32) * sig_full
    snap = torch.randn((N, total), generator=g, device=device, dtype=torch.float32) * sig_full
    mu = torch.zeros(total, device=device, dtype=torch.float32)
    for _ in range(N):
        mu += torch.randn(total, generator=g, device=device, dtype=torch.float32) * sig_full
    mu /= N
    return cur, snap, mu, offs
