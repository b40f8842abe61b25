"""Seeded synthetic inputs shared by the CUDA path, the oracle tests and the benchmark.

Holds none of the method's arithmetic: only a counter-based integer hash, textures,
sprites, camera paths and Gaussian K/V.  The five workloads mirror the structure of
the paper's clips (static scenes, slow pans, action; Sec. IV-A) at the LLaVA-1.6
token geometry (336x336 frames, 24x24 patches of 14 px; Sec. II-A).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 26021423
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_GOLD = np.uint64(0x9E3779B97F4A7C15)


def hash_u64(seed: int, stream: int, idx) -> np.ndarray:
    """Counter-based 64-bit mix of (seed, stream, index)."""
    with np.errstate(over="ignore"):
        x = np.asarray(idx, dtype=np.uint64) * _GOLD
        x = x + np.uint64(seed & 0xFFFFFFFFFFFFFFFF) * _M1 + np.uint64(stream & 0xFFFFFFFFFFFFFFFF) * _M2
        x ^= x >> np.uint64(30)
        x *= _M1
        x ^= x >> np.uint64(27)
        x *= _M2
        x ^= x >> np.uint64(31)
    return x


def uniform01(seed: int, stream: int, idx) -> np.ndarray:
    return (hash_u64(seed, stream, idx) >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def normal(seed: int, stream: int, n: int, start: int = 0) -> np.ndarray:
    """n standard normal samples (Box-Muller on two hashed uniforms per sample)."""
    i = np.arange(start, start + n, dtype=np.uint64)
    u1 = uniform01(seed, 2 * stream, i)
    u2 = uniform01(seed, 2 * stream + 1, i)
    return np.sqrt(-2.0 * np.log(1.0 - u1)) * np.cos(2.0 * np.pi * u2)


def _lattice(seed: int, stream: int, gy, gx) -> np.ndarray:
    return uniform01(seed, stream, gy.astype(np.uint64) * np.uint64(1000003) + gx.astype(np.uint64))


def _octave(seed: int, stream: int, H: int, W: int, cell: int) -> np.ndarray:
    y = np.arange(H)[:, None] / cell
    x = np.arange(W)[None, :] / cell
    y0, x0 = np.floor(y).astype(np.int64), np.floor(x).astype(np.int64)
    fy, fx = y - y0, x - x0
    fy = fy * fy * (3 - 2 * fy)
    fx = fx * fx * (3 - 2 * fx)
    v00 = _lattice(seed, stream, y0 + 0 * x0, x0 + 0 * y0)
    v01 = _lattice(seed, stream, y0 + 0 * x0, x0 + 1 + 0 * y0)
    v10 = _lattice(seed, stream, y0 + 1 + 0 * x0, x0 + 0 * y0)
    v11 = _lattice(seed, stream, y0 + 1 + 0 * x0, x0 + 1 + 0 * y0)
    return (v00 * (1 - fx) + v01 * fx) * (1 - fy) + (v10 * (1 - fx) + v11 * fx) * fy


def texture(seed: int, H: int, W: int) -> np.ndarray:
    """3-channel value noise, two octaves (32 px amplitude 1, 8 px amplitude 1/2), in [32, 224]."""
    out = np.empty((H, W, 3), np.uint8)
    for c in range(3):
        v = (_octave(seed, 10 + c, H, W, 32) + 0.5 * _octave(seed, 20 + c, H, W, 8)) / 1.5
        out[:, :, c] = np.clip(np.rint(32 + 192 * v), 0, 255).astype(np.uint8)
    return out


@dataclass
class Sprite:
    size: int
    p0: tuple
    v: tuple
    color: tuple

    def draw(self, frame: np.ndarray, t: int) -> None:
        H, W, _ = frame.shape
        pos = []
        for p, vel, lim in ((self.p0[0], self.v[0], H - self.size), (self.p0[1], self.v[1], W - self.size)):
            q = p + vel * t
            period = 2 * lim if lim > 0 else 1
            q = q % period
            pos.append(int(np.floor(period - q if q > lim else q)))
        y, x = pos
        yy, xx = np.mgrid[0:self.size, 0:self.size]
        checker = (((yy // 8) + (xx // 8)) % 2).astype(bool)
        col = np.array(self.color, np.int32)
        alt = np.clip(col - 100 * np.sign(col - 127), 0, 255)
        frame[y:y + self.size, x:x + self.size] = np.where(checker[:, :, None], alt, col).astype(np.uint8)


def _sprites(seed: int, n: int, H: int, W: int, smin: int, smax: int, vmax: float) -> list:
    out = []
    for k in range(n):
        u = uniform01(seed, 50 + k, np.arange(8))
        size = int(smin + np.floor(u[0] * (smax - smin + 1)))
        p0 = (float(u[1] * (H - size)), float(u[2] * (W - size)))
        v = (float((2 * u[3] - 1) * vmax), float((2 * u[4] - 1) * vmax))
        color = tuple(int(c) for c in np.where(u[5:8] > 0.5, 230, 25))
        out.append(Sprite(size, p0, v, color))
    return out


@dataclass
class Workload:
    """One of the five synthetic workloads."""
    index: int
    T: int
    H: int
    W: int
    n_images: int          # 1, or 5 for the anyres layout (base + 2x2 tiles)
    L: int
    heads: int = 32
    head_dim: int = 128
    background: str = "int8"   # "int8" | "int4"
    outlier_frac: float = 0.0
    outlier_mult: float = 8.0
    budget_bytes: int = 0
    description: str = ""
    seed: int = field(default=BASE_SEED)

    @property
    def n_tok(self) -> int:
        return self.n_images * (336 // 14) ** 2

    @property
    def HD(self) -> int:
        return self.heads * self.head_dim


WORKLOADS = {
    1: Workload(1, 8, 336, 336, 1, 1, background="int8",
                description="8 frames 336x336, static 0-3 then pan +2 px/frame, one 64x64 sprite, noise sigma 2; L=1"),
    2: Workload(2, 64, 336, 336, 1, 32, background="int8", outlier_frac=0.01,
                description="64 frames 336x336, fixed texture + 3 sprites (32-96 px, 0-4 px/frame); L=32, 1% x8 outliers"),
    3: Workload(3, 300, 336, 336, 1, 32, background="int4",
                description="300 frames 336x336, 120 pan 3 px/frame then 180 static with 2 sprites; L=32, int4 background"),
    4: Workload(4, 120, 672, 672, 5, 32, background="int8",
                description="120 frames 672x672 anyres (2880 tokens), scene cut every 30 frames, brightness jitter +-5; L=32"),
    5: Workload(5, 1800, 336, 336, 1, 8, background="int4", budget_bytes=40 * 10**9,
                description="1800 frames 336x336 streamed, 300-frame segments static / pan 1 / pan 8 px/frame; L=8, 40 GB budget"),
}


def thresholds(background: str) -> dict:
    """Eq. 8 thresholds.  The paper prints none; the four-tier values were set once, with the oracle, so that
    the stored tokens of workload 2 split near the paper's FP16 : INT8 : INT4 : prune proportions (Fig. 3).
    The two-tier workloads (salient FP16 + INT8 or INT4 background) keep tau_high and collapse the rest."""
    if background == "int8":
        return dict(tau_high=0.40, tau_med=-1.0, tau_low=-1.0)
    if background == "int4":
        return dict(tau_high=0.40, tau_med=0.40, tau_low=-1.0)
    if background == "four":
        return dict(tau_high=0.40, tau_med=0.36, tau_low=0.25)
    raise ValueError(background)


def frames(index: int, T: int | None = None, t0: int = 0) -> np.ndarray:
    """uint8 frames [T][H][W][3] of workload `index`, frames t0 .. t0+T-1."""
    wl = WORKLOADS[index]
    T = wl.T - t0 if T is None else T
    seed = BASE_SEED + index
    H, W = wl.H, wl.W
    out = np.empty((T, H, W, 3), np.uint8)
    if index == 1:
        canvas = texture(seed, H, W + 2 * wl.T)
        spr = [Sprite(64, (40.0, 30.0), (1.5, 2.5), (235, 40, 40))]
        for i in range(T):
            t = t0 + i
            off = 2 * max(0, t - 3)
            fr = canvas[:, off:off + W].copy()
            spr[0].draw(fr, t)
            noise = np.rint(2.0 * normal(seed, 100 + t, H * W * 3)).reshape(H, W, 3)
            out[i] = np.clip(fr.astype(np.int32) + noise.astype(np.int32), 0, 255).astype(np.uint8)
    elif index == 2:
        canvas = texture(seed, H, W)
        spr = _sprites(seed, 3, H, W, 32, 96, 4.0)
        for i in range(T):
            fr = canvas.copy()
            for s in spr:
                s.draw(fr, t0 + i)
            out[i] = fr
    elif index == 3:
        canvas = texture(seed, H, W + 3 * 120)
        spr = _sprites(seed, 2, H, W, 32, 96, 4.0)
        for i in range(T):
            t = t0 + i
            off = 3 * min(t, 119)
            fr = canvas[:, off:off + W].copy()
            if t >= 120:
                for s in spr:
                    s.draw(fr, t - 120)
            out[i] = fr
    elif index == 4:
        cache = {}
        for i in range(T):
            t = t0 + i
            scene = t // 30
            if scene not in cache:
                cache = {scene: texture(seed + 1000 * (scene + 1), H, W)}
            jit = int(np.floor(uniform01(seed, 77, np.array([t]))[0] * 11)) - 5
            out[i] = np.clip(cache[scene].astype(np.int32) + jit, 0, 255).astype(np.uint8)
    elif index == 5:
        kinds = (np.floor(uniform01(seed, 5, np.arange(6)) * 3)).astype(int)
        kinds[0], kinds[1], kinds[2] = 0, 1, 2       # every kind occurs at least once
        speed = np.array([0, 1, 8])[kinds]
        total = int((speed * 300).sum())
        canvas = texture(seed, H, W + total)
        seg_start = np.concatenate([[0], np.cumsum(speed * 300)])
        for i in range(T):
            t = t0 + i
            seg, k = divmod(t, 300)
            off = int(seg_start[seg] + speed[seg] * k)
            out[i] = canvas[:, off:off + W]
    else:
        raise ValueError(index)
    return out


def kv_numpy(index: int, frame: int, L: int | None = None, n_tok: int | None = None) -> tuple:
    """fp16 K, V [L][n_tok][HD] ~ N(0,1) for one frame (host generator, small cases)."""
    wl = WORKLOADS[index]
    L = wl.L if L is None else L
    n_tok = wl.n_tok if n_tok is None else n_tok
    n = L * n_tok * wl.HD
    seed = BASE_SEED + 100 + index
    out = []
    for kv in range(2):
        x = normal(seed, 1000 + 2 * frame + kv, n)
        if wl.outlier_frac > 0:
            u = uniform01(seed, 5000 + 2 * frame + kv, np.arange(n, dtype=np.uint64))
            x = np.where(u < wl.outlier_frac, x * wl.outlier_mult, x)
        out.append(x.astype(np.float16).reshape(L, n_tok, wl.HD))
    return out[0], out[1]


def kv_torch(index: int, frame: int, device, L: int | None = None, n_tok: int | None = None):
    """fp16 K, V [L][n_tok][HD] ~ N(0,1) for one frame, generated on `device` from the seed
    (large cases; the bytes are copied to the host for the oracle when sampled)."""
    import torch
    wl = WORKLOADS[index]
    L = wl.L if L is None else L
    n_tok = wl.n_tok if n_tok is None else n_tok
    g = torch.Generator(device=device)
    g.manual_seed(BASE_SEED + 100 + index + 7919 * (frame + 1))
    out = []
    for kv in range(2):
        x = torch.randn((L, n_tok, wl.HD), generator=g, device=device, dtype=torch.float32)
        if wl.outlier_frac > 0:
            m = torch.rand((L, n_tok, wl.HD), generator=g, device=device) < wl.outlier_frac
            x = torch.where(m, x * wl.outlier_mult, x)
        out.append(x.to(torch.float16))
    return out[0], out[1]
