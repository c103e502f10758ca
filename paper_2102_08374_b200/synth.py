"""Seeded synthetic inputs shaped like the IntSGD paper's workloads.

Input generation only -- none of the method's arithmetic lives here.  The same arrays are handed
to the CUDA library and to the CPU oracle by the tests and the benchmark.  The paper trains
ResNet18 on CIFAR-10, a 3-layer LSTM on Wikitext-2 (Section 5.1) and l2-regularised logistic
regression on LibSVM sets (Appendix C.5); none of those data are used here, only the vector
lengths, worker counts and rough value scales.

Host generators use numpy ``default_rng`` (PCG64); the ``*_device`` generators use a seeded torch
CUDA generator for vectors too large to draw on the host in reasonable time.
"""
from __future__ import annotations

import numpy as np

# ResNet-18 (CIFAR variant: 3x3 stem, no max-pool, 10 classes) parameter tensors in order:
# conv / bn-weight / bn-bias triples, the three 1x1 shortcut convs with their bn, and the
# linear layer.  62 segments, 11,173,962 parameters.
RESNET18_SEGMENTS = (
    [1728, 64, 64]
    + [36864, 64, 64] * 4
    + [73728, 128, 128, 147456, 128, 128, 8192, 128, 128] + [147456, 128, 128] * 2
    + [294912, 256, 256, 589824, 256, 256, 32768, 256, 256] + [589824, 256, 256] * 2
    + [1179648, 512, 512, 2359296, 512, 512, 131072, 512, 512] + [2359296, 512, 512] * 2
    + [5120, 10]
)
RESNET18_D = 11_173_962
assert len(RESNET18_SEGMENTS) == 62 and sum(RESNET18_SEGMENTS) == RESNET18_D


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = b + (((b >> 16) & 1) + np.uint32(0x7FFF))
    return (rounded >> 16).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


# ------------------------------------------------------------------------------------------
# Config 1: operator check.  n = 4, d = 2^20, one step from given x^0 and x^{-1}.
# ------------------------------------------------------------------------------------------
def operator_check(n: int = 4, d: int = 1 << 20):
    rng = np.random.default_rng(0)
    grads = [rng.normal(0.0, 1e-2, d).astype(np.float32) for _ in range(n)]
    rng = np.random.default_rng(1)
    x_prev = rng.normal(0.0, 1.0, d).astype(np.float32)
    x0 = (x_prev + rng.normal(0.0, 1e-3, d).astype(np.float32)).astype(np.float32)
    return dict(n=n, d=d, grads=grads, x_prev=x_prev, x0=x0, eta=0.1, beta=0.9, eps=1e-8)


# ------------------------------------------------------------------------------------------
# Config 2: l2-regularised logistic regression with heterogeneous workers (stands in for the
# LibSVM experiment).  The gradient is the user's model, computed here and given to both sides.
# ------------------------------------------------------------------------------------------
class LogisticProblem:
    def __init__(self, n: int = 16, m: int = 2048, d: int = 4096, lam: float = 1e-4, device=None):
        import torch
        self.n, self.m, self.d, self.lam = n, m, d, lam
        self.device = device or "cpu"
        w_star = np.random.default_rng(99).normal(0.0, 1.0, d).astype(np.float32)
        self.A, self.b = [], []
        for i in range(n):
            A = np.random.default_rng(100 + i).normal(0.0, 1.0, (m, d)).astype(np.float32)
            b = np.sign(A @ w_star).astype(np.float32)
            b[b == 0] = 1.0
            self.A.append(torch.from_numpy(A).to(self.device))
            self.b.append(torch.from_numpy(b).to(self.device))

    def gradients(self, x):
        """Full local gradients of f_i(x) = (1/m) sum_l log(1 + exp(-b_l a_l^T x)) + (lam/2)|x|^2."""
        import torch
        out = []
        for A, b in zip(self.A, self.b):
            z = (A @ x) * b
            s = -b * torch.sigmoid(-z)
            out.append(((A.t() @ s) / self.m + self.lam * x).contiguous())
        return out


# ------------------------------------------------------------------------------------------
# Config 3: ResNet-18-shaped flat gradient, per-layer scales log-uniform in [1e-4, 1e-1].
# ------------------------------------------------------------------------------------------
def resnet18_layer_scales() -> np.ndarray:
    return (10.0 ** np.random.default_rng(300).uniform(-4.0, -1.0, len(RESNET18_SEGMENTS))).astype(np.float32)


def resnet18_gradient(worker: int, pool_index: int = 0, segments=RESNET18_SEGMENTS) -> np.ndarray:
    scales = resnet18_layer_scales()
    rng = np.random.default_rng(301 + 100 * pool_index + worker)
    parts = [rng.standard_normal(sz, dtype=np.float32) * s for sz, s in zip(segments, scales)]
    return np.concatenate(parts).astype(np.float32)


# ------------------------------------------------------------------------------------------
# Config 4: LSTM-language-model-shaped bf16 gradient: the first 40 % of the coordinates (the
# embedding) heavy-tailed Student-t(3) * 1e-3, the rest N(0, 1e-3^2).
# ------------------------------------------------------------------------------------------
def lstm_gradient_bf16(worker: int, d: int = 1 << 25, pool_index: int = 0) -> np.ndarray:
    rng = np.random.default_rng(401 + 100 * pool_index + worker)
    k = (d * 2) // 5
    emb = rng.standard_t(3.0, k).astype(np.float32) * np.float32(1e-3)
    rest = rng.standard_normal(d - k, dtype=np.float32) * np.float32(1e-3)
    return to_bf16_bits(np.concatenate([emb, rest]))


def lstm_eta(step: int) -> float:
    """Learning rate 1.25 x 16 workers, multiplied by 0.25 at step 100."""
    return 20.0 if step < 100 else 5.0


# ------------------------------------------------------------------------------------------
# Config 5: large-model bucket sweep, g ~ N(0, 1e-3^2) fp32.
# ------------------------------------------------------------------------------------------
def bucket_gradient(worker: int, d: int, seed_base: int = 500) -> np.ndarray:
    rng = np.random.default_rng(seed_base + worker)
    return rng.standard_normal(d, dtype=np.float32) * np.float32(1e-3)


def iterate(d: int, seed: int = 7) -> np.ndarray:
    return np.random.default_rng(seed).standard_normal(d, dtype=np.float32)


def bucket_gradients_device(n: int, d: int, device, seed_base: int = 500, dtype=None):
    """n gradient vectors N(0, 1e-3^2) drawn on the device (seeded torch generator)."""
    import torch
    out = []
    for i in range(n):
        g = torch.Generator(device=device)
        g.manual_seed(seed_base + i)
        v = torch.randn(d, generator=g, device=device, dtype=torch.float32).mul_(1e-3)
        out.append(v if dtype is None else v.to(dtype))
    return out


def iterate_device(d: int, device, seed: int = 7):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return torch.randn(d, generator=g, device=device, dtype=torch.float32)
