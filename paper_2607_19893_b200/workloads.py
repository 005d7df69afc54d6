"""Seeded synthetic workloads shaped like the paper's evaluation scenes.

This module only draws random inputs (primitive attributes, cameras, target
images).  It holds none of the rendering / optimiser arithmetic, so both the
CPU oracle and the CUDA path can be fed from it without sharing any of the
method's code.  Everything is NumPy on the host; every draw comes from
``numpy.random.default_rng(1000 * cfg + purpose)``.

Five presets follow the benchmark configurations:

  1  1,024 splats, SH degree 0, one 64x64 pinhole camera at the origin
  2  100k splats, SH3, Gaussian blob, 8 orbit cameras, 256x256
  3  1M splats, SH3, unbounded 360-degree shape, 32 ring cameras, 1600x1066
  4  5M splats, SH3, same shape with larger splats, 64 cameras, 1920x1080
  5  20M splats, SH3, city blocks, 64 aerial + 64 street cameras, 1920x1080

(3 and 4 stand in for unbounded 360-degree captures, 5 for an aerial+street
city capture; no dataset item is reproduced.)
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import numpy as np

# value of the constant (degree-0) real spherical harmonic, used only to turn a
# drawn RGB colour into the stored DC coefficient: dc = (rgb - 0.5) / SH_DC
SH_DC = 0.28209479177387814


@dataclasses.dataclass
class Camera:
    width: int
    height: int
    fx: float
    fy: float
    cx: float
    cy: float
    znear: float
    zfar: float
    w2c: np.ndarray  # [3,4] float64 row-major [R|t]; +z forward, x right, y down
    bg: np.ndarray  # [3] float64

    def as_f64(self) -> np.ndarray:
        """Flat float64[23]: W,H,fx,fy,cx,cy,znear,zfar,w2c[12],bg[3]."""
        return np.concatenate(
            [
                np.array(
                    [self.width, self.height, self.fx, self.fy, self.cx, self.cy, self.znear, self.zfar],
                    dtype=np.float64,
                ),
                np.asarray(self.w2c, dtype=np.float64).reshape(12),
                np.asarray(self.bg, dtype=np.float64).reshape(3),
            ]
        )


@dataclasses.dataclass
class Scene:
    sh_degree: int
    means: np.ndarray  # [N,3] f32
    log_scales: np.ndarray  # [N,3] f32
    quats: np.ndarray  # [N,4] f32 (w,x,y,z), not necessarily unit
    opacity_logit: np.ndarray  # [N] f32
    sh: np.ndarray  # [N,K,3] f32, K=(deg+1)^2

    @property
    def n(self) -> int:
        return int(self.means.shape[0])

    @property
    def sh_k(self) -> int:
        return (self.sh_degree + 1) ** 2

    @property
    def floats_per_primitive(self) -> int:
        return 11 + 3 * self.sh_k

    def copy(self) -> "Scene":
        return Scene(
            self.sh_degree,
            self.means.copy(),
            self.log_scales.copy(),
            self.quats.copy(),
            self.opacity_logit.copy(),
            self.sh.copy(),
        )

    def astype(self, dt) -> "Scene":
        return Scene(
            self.sh_degree,
            self.means.astype(dt),
            self.log_scales.astype(dt),
            self.quats.astype(dt),
            self.opacity_logit.astype(dt),
            self.sh.astype(dt),
        )

    def zeros_like(self) -> "Scene":
        return Scene(
            self.sh_degree,
            np.zeros_like(self.means),
            np.zeros_like(self.log_scales),
            np.zeros_like(self.quats),
            np.zeros_like(self.opacity_logit),
            np.zeros_like(self.sh),
        )


@dataclasses.dataclass
class Workload:
    cfg: int
    name: str
    scene: Scene
    cameras: List[Camera]
    steps: int
    lr: np.ndarray  # [6] mean, scale, quat, opacity, sh_dc, sh_rest
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-15
    conflict_window: Optional[int] = None  # None: all pairs; k: previous k views
    seed_base: int = 0

    def target(self, view: int) -> np.ndarray:
        """Seeded uniform[0,1] target image [3,H,W] f32 for a view."""
        cam = self.cameras[view]
        rng = np.random.default_rng(self.seed_base + 500 + view)
        return rng.random((3, cam.height, cam.width), dtype=np.float32)


def look_at(eye, target, up=(0.0, 0.0, 1.0)) -> np.ndarray:
    """World-to-camera [R|t] for a camera at `eye` looking at `target`.

    Camera axes: x right, y down, z forward (rows of R).
    """
    eye = np.asarray(eye, dtype=np.float64)
    f = np.asarray(target, dtype=np.float64) - eye
    f /= np.linalg.norm(f)
    right = np.cross(f, np.asarray(up, dtype=np.float64))
    right /= np.linalg.norm(right)
    down = np.cross(f, right)
    R = np.stack([right, down, f])
    t = -R @ eye
    return np.concatenate([R, t[:, None]], axis=1)


def pose_from_yaw_pitch(eye, yaw, pitch) -> np.ndarray:
    """[R|t] for a z-up world: heading `yaw` about z, `pitch` radians above the horizon."""
    f = np.array([np.cos(pitch) * np.cos(yaw), np.cos(pitch) * np.sin(yaw), np.sin(pitch)])
    return look_at(eye, np.asarray(eye, dtype=np.float64) + f)


def _unit_vectors(rng, n):
    v = rng.standard_normal((n, 3))
    v /= np.linalg.norm(v, axis=1, keepdims=True)
    return v


def _attributes(rng, n, sh_degree, ls_mu, ls_sigma):
    k = (sh_degree + 1) ** 2
    log_scales = (ls_mu + ls_sigma * rng.standard_normal((n, 3), dtype=np.float32)).astype(np.float32)
    q = rng.standard_normal((n, 4), dtype=np.float32)
    q /= np.linalg.norm(q, axis=1, keepdims=True)
    logits = rng.standard_normal(n, dtype=np.float32)
    sh = np.empty((n, k, 3), dtype=np.float32)
    if k > 1:
        # drawn in place, slab by slab, to bound peak memory and time on the 20M preset
        step = 1 << 20
        for s in range(0, n, step):
            slab = sh[s:min(n, s + step)]
            rng.standard_normal(out=slab, dtype=np.float32)
            slab *= np.float32(0.1)
    rgb = rng.random((n, 3), dtype=np.float32)
    sh[:, 0, :] = (rgb - 0.5) / np.float32(SH_DC)
    return log_scales, q.astype(np.float32), logits, sh


def _camera(w, h, f, w2c, znear=0.2, zfar=1.0e9, bg=(0.0, 0.0, 0.0)) -> Camera:
    return Camera(w, h, float(f), float(f), w / 2.0, h / 2.0, znear, zfar, np.asarray(w2c), np.asarray(bg, dtype=np.float64))


def _ring_cameras(n_cam, radius, height, w, h, f, phase=0.0):
    cams = []
    for i in range(n_cam):
        a = phase + 2.0 * np.pi * i / n_cam
        eye = np.array([radius * np.cos(a), radius * np.sin(a), height])
        cams.append(_camera(w, h, f, look_at(eye, (0.0, 0.0, 0.0))))
    return cams


def _unbounded_means(rng, n):
    """70 % uniform in the unit ball, 30 % on a shell of radius U[3,20]; shuffled."""
    n_core = int(round(0.7 * n))
    core = _unit_vectors(rng, n_core) * np.cbrt(rng.random((n_core, 1)))
    shell = _unit_vectors(rng, n - n_core) * rng.uniform(3.0, 20.0, (n - n_core, 1))
    means = np.concatenate([core, shell]).astype(np.float32)
    rng.shuffle(means, axis=0)
    return means


DEFAULT_LR = np.full(6, 1e-3, dtype=np.float32)


def make_workload(cfg: int, n: Optional[int] = None, n_cameras: Optional[int] = None,
                  resolution: Optional[tuple] = None, city_grid: Optional[int] = None) -> Workload:
    """Build preset `cfg` (1..5).  `n`, `n_cameras`, `resolution=(W,H)` scale it down for tests;
    focal length scales with the width so the field of view is kept."""
    seed = 1000 * cfg
    rng = np.random.default_rng(seed + 1)

    def res(w, h, f):
        if resolution is None:
            return w, h, f
        return resolution[0], resolution[1], f * resolution[0] / w

    if cfg == 1:
        n = n or 1024
        means = np.stack(
            [rng.uniform(-1, 1, n), rng.uniform(-1, 1, n), rng.uniform(2, 6, n)], axis=1
        ).astype(np.float32)
        ls, q, lo, sh = _attributes(rng, n, 0, -3.0, 0.3)
        w, h, f = res(64, 64, 64.0)
        w2c = np.concatenate([np.eye(3), np.zeros((3, 1))], axis=1)
        cams = [_camera(w, h, f, w2c)]
        return Workload(1, "cfg1_1k_sh0_64x64", Scene(0, means, ls, q, lo, sh), cams, 1, DEFAULT_LR.copy(), seed_base=seed)
    if cfg == 2:
        n = n or 100_000
        means = (2.0 * rng.standard_normal((n, 3))).astype(np.float32)
        ls, q, lo, sh = _attributes(rng, n, 3, -3.0, 0.3)
        w, h, f = res(256, 256, 256.0)
        cams = _ring_cameras(n_cameras or 8, 6.0, 0.0, w, h, f)
        return Workload(2, "cfg2_100k_sh3_256x256", Scene(3, means, ls, q, lo, sh), cams, 10, DEFAULT_LR.copy(), seed_base=seed)
    if cfg == 3:
        n = n or 1_000_000
        means = _unbounded_means(rng, n)
        ls, q, lo, sh = _attributes(rng, n, 3, -5.0, 0.5)
        w, h, f = res(1600, 1066, 1400.0)
        cams = _ring_cameras(n_cameras or 32, 1.0, 0.2, w, h, f)
        return Workload(3, "cfg3_1m_sh3_1600x1066", Scene(3, means, ls, q, lo, sh), cams, 100, DEFAULT_LR.copy(), seed_base=seed)
    if cfg == 4:
        n = n or 5_000_000
        means = _unbounded_means(rng, n)
        ls, q, lo, sh = _attributes(rng, n, 3, -4.0, 0.5)
        w, h, f = res(1920, 1080, 1600.0)
        cams = _ring_cameras(n_cameras or 64, 0.45, 0.09, w, h, f)
        return Workload(4, "cfg4_5m_sh3_1920x1080", Scene(3, means, ls, q, lo, sh), cams, 64, DEFAULT_LR.copy(),
                        conflict_window=4, seed_base=seed)
    if cfg == 5:
        grid, pitch_m = 64, 30.0
        if city_grid is not None:
            # a smaller city at the SAME density per block (what a camera sees is unchanged): used for profiler
            # captures, which must keep only a few GB on the device
            grid = int(city_grid)
            n = n or int(round(20_000_000 * (grid / 64.0) ** 2))
        n = n or 20_000_000
        # per-block Poisson counts, rescaled to sum to n; primitives are stored block by block
        counts = rng.poisson(n / (grid * grid), grid * grid).astype(np.int64)
        diff = n - int(counts.sum())
        counts[: abs(diff)] += 1 if diff > 0 else -1
        counts = np.maximum(counts, 0)
        counts[-1] += n - int(counts.sum())
        block = np.repeat(np.arange(grid * grid), counts)
        bx = (block % grid).astype(np.float64)
        by = (block // grid).astype(np.float64)
        extent = grid * pitch_m
        cxm = (bx + 0.5) * pitch_m - extent / 2
        cym = (by + 0.5) * pitch_m - extent / 2
        cap = rng.uniform(0.0, 40.0, grid * grid)[block]
        means = np.stack(
            [cxm + rng.uniform(-12, 12, n), cym + rng.uniform(-12, 12, n), cap * rng.random(n)], axis=1
        ).astype(np.float32)
        ls, q, lo, sh = _attributes(rng, n, 3, float(np.log(0.3)), 0.5)
        w, h, f = res(1920, 1080, 1000.0)
        n_cam = n_cameras or 128
        n_air = n_cam // 2
        cams = []
        crng = np.random.default_rng(seed + 2)
        side = int(np.ceil(np.sqrt(n_air)))
        for i in range(n_air):  # lawn-mower grid at 150 m, pitched 60 degrees down, varied heading
            gx, gy = i % side, i // side
            if gy % 2:
                gx = side - 1 - gx
            ex = (gx + 0.5) / side * extent * 0.8 - extent * 0.4
            ey = (gy + 0.5) / side * extent * 0.8 - extent * 0.4
            yaw = crng.uniform(0, 2 * np.pi)
            cams.append(_camera(w, h, f, pose_from_yaw_pitch((ex, ey, 150.0), yaw, np.deg2rad(-60.0)), zfar=2000.0))
        for i in range(n_cam - n_air):  # street level on the street centre-lines between blocks
            line = crng.integers(1, grid)
            along = crng.uniform(-extent * 0.45, extent * 0.45)
            street = line * pitch_m - extent / 2
            if i % 2:
                eye, yaw = (street, along, 1.7), crng.choice([0.5 * np.pi, 1.5 * np.pi])
            else:
                eye, yaw = (along, street, 1.7), crng.choice([0.0, np.pi])
            cams.append(_camera(w, h, f, pose_from_yaw_pitch(eye, yaw, 0.0), zfar=400.0))
        # interleave aerial and street views so a run of steps mixes both kinds
        order = [c for pair in zip(cams[:n_air], cams[n_air:]) for c in pair] + cams[2 * min(n_air, n_cam - n_air):]
        return Workload(5, "cfg5_20m_sh3_city_1920x1080", Scene(3, means, ls, q, lo, sh), order, 50,
                        DEFAULT_LR.copy(), seed_base=seed)
    raise ValueError(f"unknown cfg {cfg}")


def tiny_scene(seed: int, n: int, sh_degree: int, width: int = 32, height: int = 32, f: float = 40.0,
               ls_mu: float = -1.6, depth=(3.0, 5.0), spread: float = 0.8):
    """A few large, well-separated-from-thresholds splats for finite-difference checks (float64)."""
    rng = np.random.default_rng(seed)
    means = np.stack(
        [rng.uniform(-spread, spread, n), rng.uniform(-spread, spread, n), rng.uniform(depth[0], depth[1], n)], axis=1
    )
    k = (sh_degree + 1) ** 2
    ls = ls_mu + 0.3 * rng.standard_normal((n, 3))
    q = rng.standard_normal((n, 4))
    lo = rng.uniform(-1.0, 1.5, n)
    sh = np.zeros((n, k, 3))
    sh[:, 0, :] = (rng.uniform(0.2, 0.9, (n, 3)) - 0.5) / SH_DC
    if k > 1:
        sh[:, 1:, :] = 0.15 * rng.standard_normal((n, k - 1, 3))
    yaw = 0.1
    eye = np.array([0.15, -0.1, -0.3])
    w2c = look_at(eye, (0.0, 0.05, 4.0), up=(np.sin(yaw), -np.cos(yaw), 0.0))
    cam = _camera(width, height, f, w2c, bg=(0.1, 0.2, 0.3))
    return Scene(sh_degree, means, ls, q, lo, sh), cam
