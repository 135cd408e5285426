"""Workload shapes for the VScan reduction path.

Only shapes and counts live here: no arithmetic of the method.  The five named
workloads follow the paper's model shapes (576 / 2880 / 16384 visual tokens,
Sec. 5.1 "Models"; pruning layers k=16 and k=14, Sec. 5.1 "Implementation
Details") with the retention budgets of Sec. 5.1 and App. B.1.
"""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class VScanConfig:
    name: str
    config_id: int          # feeds the RNG key
    dtype: str              # "f32" | "bf16": I/O dtype of features, attention rows, q/K/V/hidden
    B: int                  # images
    C: int                  # crops (encoder instances) per image
    frames: int             # F
    grid_h: int             # patch grid rows per frame
    grid_w: int             # patch grid columns per frame
    cls: int                # 1 if a [CLS] entry precedes the patches, else 0
    D: int                  # encoder feature dim
    H: int                  # encoder heads
    win_h: int
    win_w: int
    k_w: int                # local budget per window
    k_g: int                # global budget per instance
    n_clusters: int         # feature generator: number of Gaussian clusters
    n_sys: int
    n_txt: int
    Dh: int                 # LLM hidden size
    Hq: int
    Hkv: int
    d: int                  # head dim
    k2: int                 # Stage-2 survivors per image
    pos_planes: int = 1     # 1, or 3 for three-plane rotary position ids

    @property
    def N(self) -> int:
        return self.frames * self.grid_h * self.grid_w

    @property
    def L(self) -> int:
        return self.N + self.cls

    @property
    def W(self) -> int:
        return self.frames * (self.grid_h // self.win_h) * (self.grid_w // self.win_w)

    @property
    def K1(self) -> int:
        return self.k_g + self.W * self.k_w

    @property
    def instances(self) -> int:
        return self.B * self.C

    @property
    def n_vis(self) -> int:
        return self.C * self.K1

    @property
    def S(self) -> int:
        return self.n_sys + self.n_vis + self.n_txt

    @property
    def S_out(self) -> int:
        return self.S - self.n_vis + self.k2

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def with_(self, **kw) -> "VScanConfig":
        return replace(self, **kw)


_LLAVA = dict(frames=1, grid_h=24, grid_w=24, cls=1, D=1024, H=16, win_h=6, win_w=6,
              n_sys=35, Dh=4096, Hq=32, Hkv=32, d=128)

CONFIGS = {
    0: VScanConfig(name="llava15_b1_f32", config_id=0, dtype="f32", B=1, C=1, k_w=2, k_g=32,
                   n_clusters=16, n_txt=40, k2=32, **_LLAVA),
    1: VScanConfig(name="llava15_b256_bf16", config_id=1, dtype="bf16", B=256, C=1, k_w=6, k_g=96,
                   n_clusters=16, n_txt=64, k2=96, **_LLAVA),
    2: VScanConfig(name="llavanext_b32_bf16", config_id=2, dtype="bf16", B=32, C=5, k_w=2, k_g=32,
                   n_clusters=64, n_txt=64, k2=160, **_LLAVA),
    3: VScanConfig(name="longframes_b4_bf16", config_id=3, dtype="bf16", B=4, C=1, frames=16,
                   grid_h=32, grid_w=32, cls=0, D=1280, H=16, win_h=8, win_w=8, k_w=4, k_g=1024,
                   n_clusters=64, n_sys=0, n_txt=128, Dh=3584, Hq=28, Hkv=4, d=128, k2=1024),
}

# Retention sweep at the 2880-token shape: per-crop kept count -> (k_w, k_g).
# 25 % of 2880 = 720 = 144 per crop; the local half (72) does not divide by 16
# windows, so k_w = floor(72/16) = 4 and the global scan takes the rest.
SWEEP_BUDGETS = {"25%": (4, 80), "11.1%": (2, 32), "5.5%": (1, 16)}
SWEEP_BATCHES = (1, 8, 64, 256, 512)


def sweep_config(batch: int, retention: str) -> VScanConfig:
    k_w, k_g = SWEEP_BUDGETS[retention]
    base = CONFIGS[2]
    k1 = k_g + base.W * k_w
    return base.with_(name=f"sweep_b{batch}_{retention}", config_id=4, B=batch, k_w=k_w, k_g=k_g,
                      k2=(base.C * k1) // 2)


def tiny_config(dtype: str = "f32", **kw) -> VScanConfig:
    """A shape small enough for pure-Python brute force, with several windows and GQA."""
    base = VScanConfig(name="tiny", config_id=99, dtype=dtype, B=2, C=2, frames=1, grid_h=4,
                       grid_w=6, cls=1, D=8, H=3, win_h=2, win_w=3, k_w=1, k_g=3, n_clusters=3,
                       n_sys=2, n_txt=3, Dh=16, Hq=4, Hkv=2, d=8, k2=5)
    return base.with_(**kw)
