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
    vis_in: int = 0         # visual tokens entering Stage 2 when that is not C * K1 (schedules without Stage 1)

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
        return self.vis_in if self.vis_in > 0 else self.C * self.K1

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


def _split_budget(base: VScanConfig, kept: int, local_share: float):
    """(k_w, k_g) for `kept` tokens per crop with `local_share` of them from the local scan: the per-window
    budget is the share divided evenly over the windows, rounded down; the global scan takes the rest, so
    the total is exact (the rule of the 25 % sweep point above)."""
    k_w = min(int(kept * local_share) // base.W, base.win_h * base.win_w)
    return k_w, kept - base.W * k_w


# (pruning layer k, R2 in percent) as printed in Table 1
TABLE1_SETTINGS = ((2, 73.3), (8, 66.7), (12, 60.0), (16, 50.0), (20, 33.3), (24, 0.0))


def schedule_points():
    """Pruning schedules of the paper as throughput workloads at the 2880-token shape (5 crops of 576
    patches, batch 32).  Only counts change; the layer index of a schedule does not change the work.
    -> list of (label, config, runs_stage1).
      Table 1: global scan only to R1 = 50 % / 25 %, then the (pruning layer k, R2) pairs the table prints
               (each pair averages 75 % of the Stage-1 set over the 32 LLM layers).
      Table 6(a): R1 / R2 pairs with the same 11.1 % average; Table 6(b): global:local share at R1 = 16.7 %.
      App. B.1: a schedule without Stage 1 that prunes all 2880 tokens to 5.2 % at an early layer."""
    base = CONFIGS[2]
    pts = []
    for r1, kept in (("50%", 288), ("25%", 144)):
        for k, r2 in TABLE1_SETTINGS:
            k2 = round(base.C * kept * r2 / 100)
            pts.append((f"table1 R1={r1} k={k}", base.with_(name=f"table1_{kept}_k{k}", config_id=5, k_w=0, k_g=kept,
                                                             k2=k2), True))
    for r1, kept, r2 in (("11.1%", 64, 1.0), ("13.3%", 77, 2 / 3), ("14.8%", 85, 0.5), ("16.7%", 96, 1 / 3),
                         ("22.2%", 128, 0.0)):
        k_w, k_g = _split_budget(base, kept, 0.5)
        pts.append((f"table6a R1={r1} R2={100 * r2:.1f}%", base.with_(name=f"table6a_{kept}", config_id=6, k_w=k_w,
                                                                      k_g=k_g, k2=round(base.C * kept * r2)), True))
    for share in (1.0, 0.75, 0.5, 0.25, 0.0):
        k_w, k_g = _split_budget(base, 96, share)
        pts.append((f"table6b global:local={100 - 100 * share:.0f}:{100 * share:.0f}",
                    base.with_(name=f"table6b_{int(100 * share)}", config_id=7, k_w=k_w, k_g=k_g, k2=base.C * 32), True))
    full = base.C * base.N
    pts.append(("appB1 no stage 1, 5.2% from an early layer",
                base.with_(name="appB1_5.2", config_id=8, vis_in=full, k2=round(0.052 * full)), False))
    return pts


def tiny_config(dtype: str = "f32", **kw) -> VScanConfig:
    """A shape small enough for pure-Python brute force, with several windows and GQA."""
    base = VScanConfig(name="tiny", config_id=99, dtype=dtype, B=2, C=2, frames=1, grid_h=4,
                       grid_w=6, cls=1, D=8, H=3, win_h=2, win_w=3, k_w=1, k_g=3, n_clusters=3,
                       n_sys=2, n_txt=3, Dh=16, Hq=4, Hkv=2, d=8, k2=5)
    return base.with_(**kw)
