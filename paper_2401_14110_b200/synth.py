"""Seeded synthetic inputs for the LBA contraction.

This module only makes inputs: random tensors with the shapes and value distributions of
the paper's workloads, and their encoding as OCP E4M3 bytes with power-free absmax scales.
It holds none of the method's arithmetic (no Q, no FMAq, no accumulation) and is the one
module that both the CUDA tests and the CPU oracle's tests draw inputs from.  The E4M3
encoding itself is PyTorch's ``float8_e4m3fn`` cast (round-to-nearest-even), applied after
clamping to the largest finite value 448.

Stand-ins: the paper evaluates on ImageNet, SQuAD and pretrained weights; none of those are
used here.  Only tensor shapes and rough value distributions (Gaussian activations, He-normal
or N(0, 0.02^2) weights, a few outlier feature columns for the transformer case) are kept.
"""
import numpy as np
import torch

E4M3_MAX = 448.0
BASE_SEED = 20240114


def seed_for(config: int, tensor_index: int) -> int:
    return BASE_SEED + 1000 * int(config) + int(tensor_index)


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def gaussian(shape, seed: int, std: float = 1.0) -> torch.Tensor:
    return torch.randn(tuple(shape), generator=_gen(seed), dtype=torch.float32) * std


def he_normal(shape, fan_in: int, seed: int) -> torch.Tensor:
    return gaussian(shape, seed, std=float(np.sqrt(2.0 / fan_in)))


def with_outlier_columns(t: torch.Tensor, seed: int, fraction: float = 0.01, gain: float = 20.0) -> torch.Tensor:
    """Multiply a seeded ``fraction`` of the last-dim features by ``gain`` (transformer-style outliers)."""
    n = t.shape[-1]
    k = max(1, int(n * fraction))
    cols = torch.randperm(n, generator=_gen(seed))[:k]
    t = t.clone()
    t[..., cols] *= gain
    return t


def e4m3_encode(t: torch.Tensor) -> torch.Tensor:
    """float32 tensor -> uint8 tensor of E4M3 codes (clamped to +-448, nearest-even)."""
    t = t.detach().to(torch.float32).clamp(-E4M3_MAX, E4M3_MAX)
    return t.to(torch.float8_e4m3fn).view(torch.uint8)


def e4m3_decode(codes: torch.Tensor) -> torch.Tensor:
    """uint8 E4M3 codes -> float32 values (PyTorch's cast; used to build inputs and glue only)."""
    return codes.view(torch.float8_e4m3fn).to(torch.float32)


M4E3_MAX = 248.0


def m4e3_encode(t: torch.Tensor) -> torch.Tensor:
    """float32 tensor -> uint8 codes of the paper's W/A byte format (s eee mmmm, magnitudes 2^e (1 + m/16), e = 0..7,
    the code e = m = 0 being zero): magnitudes are clamped to 248, rounded to the nearest grid point (ties to the even
    mantissa), and those below 1 become zero; the magnitude 1, whose code means zero, is moved up to 1.0625.
    (The paper rounds stochastically while training; this generator only has to land on the grid.)"""
    t = t.detach().to(torch.float32)
    mag = t.abs().clamp(max=M4E3_MAX)
    e = torch.floor(torch.log2(mag.clamp_min(1.0))).clamp(0, 7)
    step = torch.exp2(e) / 16.0
    q = torch.round(mag / step) * step                      # torch.round: ties to even
    e2 = torch.floor(torch.log2(q.clamp_min(1.0))).clamp(0, 7)   # rounding may have carried into the next binade
    m = torch.round(q / torch.exp2(e2) * 16.0 - 16.0).clamp(0, 15)
    code = (e2.to(torch.int32) << 4) | m.to(torch.int32)
    code = torch.where(code == 0, torch.ones_like(code), code)   # magnitude 1 -> 1.0625
    code = torch.where(mag < 1.0, torch.zeros_like(code), code)
    code = code | ((t < 0) & (code != 0)).to(torch.int32) * 0x80
    return code.to(torch.uint8)


def m4e3_decode(codes: torch.Tensor) -> torch.Tensor:
    """uint8 codes of the paper's W/A byte format -> float32 values (used to build inputs and glue only)."""
    c = codes.to(torch.int32)
    mag = torch.exp2(((c >> 4) & 7).to(torch.float32)) * (1.0 + (c & 15).to(torch.float32) / 16.0)
    mag = torch.where((c & 0x7F) == 0, torch.zeros_like(mag), mag)
    return torch.where((c & 0x80) != 0, -mag, mag)


def quantise_m4e3_per_tensor(t: torch.Tensor):
    """(codes, scale[1]) in the paper's flex-bias W/A format (Sec. 3.1): one power-of-two scale per tensor, the
    smallest that keeps the largest magnitude at or below 248 (the largest integer bias that prevents overflow)."""
    absmax = float(t.detach().abs().max())
    exp = int(np.ceil(np.log2(max(absmax, 1e-30) / M4E3_MAX)))
    if absmax / 2.0 ** exp > M4E3_MAX:
        exp += 1
    scale = torch.tensor([2.0 ** exp], dtype=torch.float32, device=t.device)
    return m4e3_encode(t / scale), scale


def quantise_per_tensor(t: torch.Tensor):
    """(codes, scale[1]) with scale = absmax/448 so the largest magnitude maps to 448."""
    absmax = t.detach().abs().max().to(torch.float32)
    scale = (absmax / E4M3_MAX).clamp_min(torch.finfo(torch.float32).tiny).reshape(1)
    return e4m3_encode(t / scale), scale


def quantise_per_channel(w: torch.Tensor):
    """(codes, scale[C]) with one absmax/448 scale per leading-dim channel."""
    flat = w.detach().reshape(w.shape[0], -1)
    absmax = flat.abs().max(dim=1).values.to(torch.float32)
    scale = (absmax / E4M3_MAX).clamp_min(torch.finfo(torch.float32).tiny)
    shape = (-1,) + (1,) * (w.dim() - 1)
    return e4m3_encode(w / scale.reshape(shape)), scale


def random_codes(shape, seed: int, include_zero_codes: bool = True) -> torch.Tensor:
    """Uniform draw over the 254 finite E4M3 codes (0x7F and 0xFF are NaN and never drawn)."""
    finite = [c for c in range(256) if (c & 0x7F) != 0x7F]
    if not include_zero_codes:
        finite = [c for c in finite if (c & 0x7F) != 0]
    table = torch.tensor(finite, dtype=torch.uint8)
    idx = torch.randint(0, len(finite), tuple(shape), generator=_gen(seed))
    return table[idx]


def small_integer_codes(shape, seed: int, max_abs: int = 8) -> torch.Tensor:
    """E4M3 codes of integers in [-max_abs, max_abs] (all exactly representable for max_abs <= 16)."""
    v = torch.randint(-max_abs, max_abs + 1, tuple(shape), generator=_gen(seed)).to(torch.float32)
    return e4m3_encode(v)


def gemm_case(M: int, N: int, K: int, config: int, outliers: bool = False, weight_std: float = 1.0):
    """A [M][K] per-tensor scaled, B [N][K] per-tensor scaled Gaussian operands as E4M3 codes."""
    a = gaussian((M, K), seed_for(config, 0))
    if outliers:
        a = with_outlier_columns(a, seed_for(config, 2))
    b = gaussian((N, K), seed_for(config, 1), std=weight_std)
    a_codes, sa = quantise_per_tensor(a)
    b_codes, sb = quantise_per_tensor(b)
    return a_codes, sa, b_codes, sb


def sample_tiles(M: int, N: int, n_tiles: int, tile: int, seed: int):
    """Seeded (m, n) index lists covering ``n_tiles`` random ``tile`` x ``tile`` output tiles."""
    g = _gen(seed)
    th, tw = min(tile, M), min(tile, N)
    m0 = torch.randint(0, M - th + 1, (n_tiles,), generator=g)
    n0 = torch.randint(0, N - tw + 1, (n_tiles,), generator=g)
    dm, dn = torch.meshgrid(torch.arange(th), torch.arange(tw), indexing="ij")
    ms = (m0[:, None, None] + dm[None]).reshape(-1)
    ns = (n0[:, None, None] + dn[None]).reshape(-1)
    return ms.numpy().astype(np.int64), ns.numpy().astype(np.int64)
