"""Seeded synthetic weight updates shaped like the paper's networks.

Input generation only: nothing here performs any step of the compression
method.  The same bytes are handed to the CUDA library and, in tests, to the
CPU checker.  The paper evaluates on trained networks (Section "Networks and
Datasets": ResNet50 on ImageNet, a two-layer 650-unit word LSTM on PTB, ...);
these generators keep the tensor shapes of those networks and draw the values
from simple distributions instead.

Seeds: ``1000 * config + 10 * round + client`` unless a caller says otherwise.
"""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple

import numpy as np

__all__ = [
    "seed_for", "resnet50_shapes", "word_lstm_shapes", "normal_flat",
    "resnet50_update", "word_lstm_update", "student_t_flat", "student_t_flat_torch",
    "adversarial_cases",
]


def seed_for(config: int, round_: int = 0, client: int = 0) -> int:
    return 1000 * config + 10 * round_ + client


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(seed))


# ---------------------------------------------------------------------------
# shapes
# ---------------------------------------------------------------------------

def resnet50_shapes() -> List[Tuple[str, Tuple[int, ...], int]]:
    """(name, shape, fan_in) for the 161 tensors of a 50-layer bottleneck ResNet.

    Built from the architecture itself: a 7x7 stem, four stages of
    [3, 4, 6, 3] bottleneck blocks of widths 64/128/256/512 (1x1, 3x3, 1x1
    with a 1x1 projection in each stage's first block), a scale and a shift
    vector after every convolution, and a 2048->1000 classifier with bias:
    53 + 106 + 2 tensors, 25 557 032 parameters.
    """
    out: List[Tuple[str, Tuple[int, ...], int]] = []

    def conv(name, cin, cout, ksz):
        out.append((name + ".w", (cout, cin, ksz, ksz), cin * ksz * ksz))
        out.append((name + ".scale", (cout,), cout))
        out.append((name + ".shift", (cout,), cout))

    conv("stem", 3, 64, 7)
    cin = 64
    for s, (width, blocks) in enumerate(zip((64, 128, 256, 512), (3, 4, 6, 3))):
        for blk in range(blocks):
            base = f"s{s}.b{blk}"
            conv(base + ".c1", cin, width, 1)
            conv(base + ".c2", width, width, 3)
            conv(base + ".c3", width, 4 * width, 1)
            if blk == 0:
                conv(base + ".proj", cin, 4 * width, 1)
            cin = 4 * width
    out.append(("fc.w", (1000, 2048), 2048))
    out.append(("fc.b", (1000,), 2048))
    return out


def word_lstm_shapes() -> List[Tuple[str, Tuple[int, ...]]]:
    """Two-layer, 650-unit word LSTM over a 10 000-word vocabulary."""
    return [
        ("embedding", (10000, 650)),
        ("lstm0.w", (1300, 2600)), ("lstm0.b", (2600,)),
        ("lstm1.w", (1300, 2600)), ("lstm1.b", (2600,)),
        ("softmax.w", (650, 10000)),
    ]


# ---------------------------------------------------------------------------
# values
# ---------------------------------------------------------------------------

def normal_flat(n: int, std: float, seed: int) -> np.ndarray:
    """n i.i.d. N(0, std^2) fp32 values."""
    return (_rng(seed).standard_normal(n, dtype=np.float32) * np.float32(std)).astype(np.float32)


def resnet50_update(seed: int) -> List[np.ndarray]:
    """One flat fp32 update per ResNet-50 tensor, N(0, (1e-2/sqrt(fan_in))^2)."""
    rng = _rng(seed)
    tensors = []
    for _, shape, fan_in in resnet50_shapes():
        n = int(np.prod(shape))
        sigma = np.float32(1e-2 / math.sqrt(fan_in))
        tensors.append(rng.standard_normal(n, dtype=np.float32) * sigma)
    return tensors


def word_lstm_update(seed: int) -> List[np.ndarray]:
    """One flat fp32 update per LSTM tensor, Laplace(0, 1e-3)."""
    rng = _rng(seed)
    return [rng.laplace(0.0, 1e-3, int(np.prod(shape))).astype(np.float32)
            for _, shape in word_lstm_shapes()]


def student_t_flat(n: int, seed: int, nu: float = 3.0, scale: float = 1e-3) -> np.ndarray:
    """n i.i.d. Student-t(nu) values times ``scale`` (heavy tails), fp32, on the host."""
    return (_rng(seed).standard_t(nu, n) * scale).astype(np.float32)


def student_t_flat_torch(n: int, seed: int, device, nu: int = 3, scale: float = 1e-3):
    """Same distribution drawn on ``device`` with torch's seeded generator.

    For sizes where host generation takes minutes.  Built in slices so the
    temporaries stay small: normal / sqrt(chi2_nu / nu), chi2 as a sum of nu
    squared normals."""
    import torch

    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    out = torch.empty(n, dtype=torch.float32, device=device)
    step = 1 << 26
    for lo in range(0, n, step):
        m = min(step, n - lo)
        z = torch.randn(m, generator=gen, device=device, dtype=torch.float32)
        chi = torch.zeros(m, device=device, dtype=torch.float32)
        for _ in range(int(nu)):
            chi += torch.randn(m, generator=gen, device=device, dtype=torch.float32) ** 2
        out[lo:lo + m] = z / torch.sqrt(chi / float(nu)) * scale
    return out


def adversarial_cases(seed: int = 7) -> List[Tuple[str, np.ndarray, np.ndarray, float]]:
    """Small (name, update, residual, p) cases that stress ties, zeros, tails and ragged sizes."""
    rng = _rng(seed)
    f32 = np.float32
    cases: List[Tuple[str, np.ndarray, np.ndarray, float]] = []

    def add(name, upd, p, res=None):
        upd = np.ascontiguousarray(upd, dtype=f32)
        res = np.zeros_like(upd) if res is None else np.ascontiguousarray(res, dtype=f32)
        cases.append((name, upd, res, p))

    add("all_zero", np.zeros(1000), 0.01)
    add("all_equal_pos", np.full(777, 0.25), 0.05)
    add("all_equal_neg", np.full(777, -0.25), 0.05)
    half = rng.standard_normal(4099).astype(f32)
    half[rng.random(4099) < 0.5] = 0.0
    add("half_zero", half, 0.3)
    pm0 = np.zeros(300, dtype=f32)
    pm0[::2] = -0.0
    add("signed_zeros", pm0, 0.1)
    spike = np.zeros(100000, dtype=f32)
    spike[99990] = 3.0
    add("single_spike_far", spike, 1e-5)
    cl = np.zeros(70000, dtype=f32)
    cl[10:20] = 1.0
    cl[69000:69010] = 1.0
    add("clustered_spikes_long_runs", cl, 20 / 70000)
    den = (rng.standard_normal(2049) * 1e-41).astype(f32)
    add("denormals", den, 0.02)
    add("n_lt_inv_p", rng.standard_normal(64).astype(f32), 0.001)
    add("n_1", np.array([-2.0]), 0.5)
    add("n_2", np.array([1.0, -1.0]), 0.5)
    add("ragged_1021", rng.standard_normal(1021).astype(f32), 0.01)
    add("ragged_4097", rng.standard_normal(4097).astype(f32) * 1e-3, 0.01)
    sym = rng.standard_normal(5000).astype(f32)
    add("symmetric_pm", np.concatenate([sym, -sym]), 0.01)
    ties = np.round(rng.standard_normal(20000) * 4).astype(f32) / 4
    add("quantised_ties", ties, 0.02)
    add("only_negative", -np.abs(rng.standard_normal(3000)).astype(f32), 0.01)
    add("few_positive", np.where(rng.random(3000) < 0.002, 1.0, -rng.random(3000)), 0.01)
    add("p_large_k_eq_n_half", rng.standard_normal(512).astype(f32), 0.5)
    add("p_0.9_overlap", rng.standard_normal(301).astype(f32), 0.9)
    add("carried_residual", rng.standard_normal(9000).astype(f32) * 1e-3, 0.01,
        res=rng.standard_normal(9000).astype(f32) * 3e-3)
    big = rng.standard_normal(6000).astype(f32)
    big[100] = 3e38
    big[200] = -3e38
    add("huge_magnitudes", big, 0.001)
    return cases
