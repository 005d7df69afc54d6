"""Pins of the oracle's binning, sort, compositing and loss against closed forms, invariants and
brute force (no GPU)."""
import numpy as np

from paper_2607_19893_b200 import workloads as wl
from test_oracle_project_pins import cam_identity, one_splat

SH_DC = 0.28209479177387814


def stack_scenes(scenes):
    return wl.Scene(
        scenes[0].sh_degree,
        np.concatenate([s.means for s in scenes]),
        np.concatenate([s.log_scales for s in scenes]),
        np.concatenate([s.quats for s in scenes]),
        np.concatenate([s.opacity_logit for s in scenes]),
        np.concatenate([s.sh for s in scenes]),
    )


def logit(o):
    return np.log(o / (1 - o))


# ------------------------------------------------------------------------------- bin / sort
def test_bin_sort_matches_bruteforce(oracle32):
    w = wl.make_workload(2, n=5000)
    cam = w.cameras[2]
    p = oracle32.project(w.scene, cam)
    keys, vals, ranges = oracle32.bin_sort(p, cam)
    tx, ty = oracle32.grid(cam)
    # brute force: enumerate (tile, primitive) pairs, order by (tile, depth bits, primitive)
    tiles, bits, prim = [], [], []
    dbits = p.depth.astype(np.float32).view(np.uint32)
    for i in np.nonzero(p.tiles_touched)[0]:
        x0, y0, x1, y1 = p.rect[i]
        for yy in range(y0, y1):
            for xx in range(x0, x1):
                tiles.append(yy * tx + xx)
                bits.append(dbits[i])
                prim.append(i)
    tiles, bits, prim = np.array(tiles, np.uint64), np.array(bits, np.uint64), np.array(prim, np.uint32)
    order = np.lexsort((prim, bits, tiles))
    assert len(keys) == len(order) == int(p.tiles_touched.sum())
    assert np.array_equal(keys, (tiles[order] << np.uint64(32)) | bits[order])
    assert np.array_equal(vals, prim[order])
    # invariants
    assert np.all(np.diff(keys.astype(np.int64)) >= 0)
    kt = (keys >> np.uint64(32)).astype(np.int64)
    pos = 0
    for t in range(tx * ty):
        s, e = ranges[t]
        cnt = int((kt == t).sum())
        assert e - s == cnt
        if cnt:
            assert s == pos and np.all(kt[s:e] == t)
        pos += cnt
    assert pos == len(keys)
    # each (tile, primitive) pair exactly once
    assert len(np.unique(kt * (1 << 32) + vals.astype(np.int64))) == len(keys)


def test_equal_depth_ties_keep_primitive_order(oracle32):
    # identical splats: identical keys per tile, values must ascend
    s = stack_scenes([one_splat((0, 0, 4.0), (-1.0,) * 3, (1, 0, 0, 0)) for _ in range(7)])
    cam = cam_identity()
    p = oracle32.project(s, cam)
    keys, vals, ranges = oracle32.bin_sort(p, cam)
    for t in range(len(ranges)):
        seg = vals[ranges[t, 0]:ranges[t, 1]]
        assert np.array_equal(seg, np.arange(7)[: len(seg)])


def test_sort_is_invariant_under_input_permutation(oracle32):
    w = wl.make_workload(1)
    cam = w.cameras[0]
    p = oracle32.project(w.scene, cam)
    keys, vals, ranges = oracle32.bin_sort(p, cam)
    perm = np.random.default_rng(3).permutation(w.scene.n)
    s2 = wl.Scene(0, w.scene.means[perm], w.scene.log_scales[perm], w.scene.quats[perm], w.scene.opacity_logit[perm],
                  w.scene.sh[perm])
    p2 = oracle32.project(s2, cam)
    keys2, vals2, ranges2 = oracle32.bin_sort(p2, cam)
    assert np.array_equal(keys, keys2) and np.array_equal(ranges, ranges2)
    # same primitives per key group (order inside equal keys may differ after renumbering)
    assert np.array_equal(np.sort(perm[vals2]), np.sort(vals))


# ------------------------------------------------------------------------------- forward
def render(o, scene, cam):
    return o.view_forward(scene, cam)


def test_single_isotropic_splat_image_closed_form(oracle64):
    # opacity 0.3 < 0.353, so alpha falls below 1/255 inside the 3-sigma square and the tile
    # rectangle never truncates a visible contribution
    f, z, s0, o = 64.0, 4.0, np.exp(-1.6), 0.3
    c, bg = np.array([0.9, 0.4, 0.2]), np.array([0.1, 0.2, 0.3])
    cam = cam_identity(bg=bg)
    scene = one_splat((0.03, -0.02, z), (-1.6,) * 3, (1, 0, 0, 0), logit(o), c)
    r = render(oracle64, scene, cam)
    t = scene.means[0]
    J = np.array([[f / z, 0, -f * t[0] / z ** 2], [0, f / z, -f * t[1] / z ** 2]])
    inv = np.linalg.inv(s0 ** 2 * J @ J.T + 0.3 * np.eye(2))
    u, v = f * t[0] / z + 32, f * t[1] / z + 32
    yy, xx = np.meshgrid(np.arange(64) + 0.5, np.arange(64) + 0.5, indexing="ij")
    dx, dy = u - xx, v - yy
    alpha = o * np.exp(-0.5 * (inv[0, 0] * dx * dx + inv[1, 1] * dy * dy) - inv[0, 1] * dx * dy)
    alpha[alpha < 1 / 255] = 0
    want = bg[:, None, None] + (c - bg)[:, None, None] * alpha[None]
    assert np.allclose(r["out"], want, atol=1e-12)
    assert np.allclose(r["final_T"], 1 - alpha, atol=1e-12)
    assert np.array_equal(r["n_contrib"], (alpha > 0).astype(np.uint32))


def test_coaxial_splats_transmittance_product(oracle64):
    ops = [0.5, 0.3, 0.6, 0.2]
    cols = np.array([[1, 0, 0], [0, 1, 0], [0, 0, 1], [1, 1, 0]], float)
    zs = [3.0, 4.0, 5.0, 6.0]
    # sub-pixel splats: the 0.3 dilation dominates, G at the pixel nearest the axis is known
    scene = stack_scenes([one_splat((0.25 * z / 64, 0.25 * z / 64, z), (-9,) * 3, (1, 0, 0, 0), logit(o), c)
                          for z, o, c in zip(zs, ops, cols)][::-1])  # stored back to front on purpose
    cam = cam_identity()
    r = render(oracle64, scene, cam)
    # centre is at pixel coordinate 32.25; pixel (32,32) is sampled at 32.5
    j = i = 32
    T, C = 1.0, np.zeros(3)
    for z, o, c in zip(zs, ops, cols):
        var = (64 * np.exp(-9) / z) ** 2 + 0.3
        a = o * np.exp(-0.5 * 2 * 0.25 ** 2 / var)
        C += c * a * T
        T *= 1 - a
    assert np.allclose(r["out"][:, j, i], C, atol=1e-9)
    assert np.isclose(r["final_T"][j, i], T, atol=1e-9)
    assert r["n_contrib"][j, i] == 4


def test_alpha_clamp_and_skip_threshold(oracle64):
    cam = cam_identity()
    # opacity 0.999 at the centre: alpha is clamped to 0.99
    hi = one_splat((0.5 * 4 / 64, 0.5 * 4 / 64, 4.0), (-1,) * 3, (1, 0, 0, 0), logit(0.999), (1, 1, 1))
    r = render(oracle64, hi, cam)
    assert np.isclose(r["final_T"][32, 32], 0.01, atol=1e-12) and np.isclose(r["out"][0, 32, 32], 0.99, atol=1e-12)
    assert r["final_T"].min() >= 0.01 - 1e-12
    # opacity just below 1/255 never contributes; just above contributes at the centre pixel only
    lo = one_splat((0.5 * 4 / 64, 0.5 * 4 / 64, 4.0), (-9,) * 3, (1, 0, 0, 0), logit(0.0039), (1, 1, 1))
    r = render(oracle64, lo, cam)
    assert np.all(r["out"] == 0) and np.all(r["final_T"] == 1) and np.all(r["n_contrib"] == 0)
    lo = one_splat((0.5 * 4 / 64, 0.5 * 4 / 64, 4.0), (-9,) * 3, (1, 0, 0, 0), logit(0.00395), (1, 1, 1))
    r = render(oracle64, lo, cam)
    assert r["n_contrib"].sum() == 1 and np.isclose(r["out"][0, 32, 32], 0.00395, atol=1e-9)


def test_termination_stops_before_crossing(oracle64):
    # eight opaque-ish layers: T after k layers = 0.3^k; 0.3^7 = 2.2e-4 is kept, the 8th would give 6.6e-5 < 1e-4
    cam = cam_identity(bg=(1, 1, 1))
    scene = stack_scenes([one_splat((0.5 * z / 64, 0.5 * z / 64, z), (-1,) * 3, (1, 0, 0, 0), logit(0.7), (0, 0, 0))
                          for z in np.linspace(3, 6, 8)])
    r = render(oracle64, scene, cam)
    assert np.isclose(r["final_T"][32, 32], 0.3 ** 7, rtol=1e-9)
    assert r["n_contrib"][32, 32] == 7
    assert np.isclose(r["out"][0, 32, 32], 0.3 ** 7, rtol=1e-9)  # background through the remaining transmittance
    assert r["final_T"].min() >= 1e-4


def test_partition_of_unity_and_invariants(oracle32):
    w = wl.make_workload(2, n=20000)
    cam = w.cameras[0]
    cam.bg = np.ones(3)
    s = w.scene.copy()
    s.sh[:] = 0
    s.sh[:, 0, :] = 0.5 / SH_DC  # every colour exactly 1
    r = render(oracle32, s, cam)
    assert np.allclose(r["out"], 1.0, atol=2e-6)
    assert r["final_T"].min() >= 1e-4 and r["final_T"].max() <= 1.0
    lens = (r["ranges"][:, 1] - r["ranges"][:, 0]).reshape(16, 16)
    assert np.all(r["n_contrib"].reshape(16, 16, 16, 16).max(axis=(1, 3)) <= lens)
    # counters: traversed entries bounded by the list, contributing pairs bounded by evaluated pairs
    c = r["counters"]
    assert c[0] <= len(r["keys"]) and c[2] <= c[1] <= 256 * len(r["keys"])


def test_transmittance_monotone_under_added_splats(oracle32):
    w = wl.make_workload(1)
    cam = w.cameras[0]
    full = render(oracle32, w.scene, cam)
    half = wl.Scene(0, *(a[:512] for a in (w.scene.means, w.scene.log_scales, w.scene.quats, w.scene.opacity_logit,
                                           w.scene.sh)))
    part = render(oracle32, half, cam)
    # adding splats can only lower the final transmittance, unless early termination kicked in
    live = full["final_T"] > 2e-4
    assert np.all(full["final_T"][live] <= part["final_T"][live] + 1e-6)


def test_edge_tiles_of_ragged_image(oracle32):
    w = wl.make_workload(2, n=3000, resolution=(100, 70))
    cam = w.cameras[0]
    r = render(oracle32, w.scene, cam)
    assert r["out"].shape == (3, 70, 100) and np.isfinite(r["out"]).all()
    assert oracle32.grid(cam) == (7, 5)


# ------------------------------------------------------------------------------- loss
def test_l1_loss_hand_value(oracle64):
    out = np.array([[[0.5, 0.2], [0.0, 1.0]], [[0.1, 0.1], [0.3, 0.9]], [[0.0, 0.0], [1.0, 1.0]]])
    tgt = np.array([[[0.25, 0.2], [0.5, 0.0]], [[0.1, 0.6], [0.3, 1.0]], [[1.0, 0.0], [0.5, 1.0]]])
    loss, g = oracle64.l1_loss(out, tgt)
    assert np.isclose(loss, (0.25 + 0.5 + 1.0 + 0.5 + 0.1 + 1.0 + 0.5) / 12)
    assert np.array_equal(g * 12, np.sign(out - tgt))
