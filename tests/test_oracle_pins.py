"""Pins for the CPU oracle: every function is checked against something other than itself --
hand-worked values (tests/golden), closed forms, invariants, special cases that reduce to a
numpy/torch library routine, and brute force on tiny inputs.  No GPU needed."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2603_05168_b200 import inputs


def _read_golden(path):
    out = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = [float(v) for v in vals]
    return out


# ------------------------------------------------------------------------------------------------
# Hand-worked example: Eq. 1-3 order, layout, and the negative control (mask-then-quant).
# ------------------------------------------------------------------------------------------------
def test_worked_example_quant_then_mask(golden_dir):
    g = _read_golden(os.path.join(golden_dir, "quant_then_mask_worked_example.txt"))
    W = np.array([g["W"]], np.float32)
    r = oracle.quantize_mask_pack(W)
    assert r["scale"] == np.float32(g["gamma"][0])
    assert r["dense_q"].tolist() == [[int(v) for v in g["dense_q"]]]
    assert r["mask"].tolist() == [[int(v) for v in g["mask"]]]
    assert r["vals"].tolist() == [[int(v) for v in g["vals"]]]
    assert r["meta"].tolist() == [[int(v) for v in g["meta"]]]
    weff, mask = oracle.unpack24(r["vals"], r["meta"])
    assert weff.tolist() == [[int(v) for v in g["weff"]]]
    # negative control: quantising the masked weights with the masked-subset gamma gives another
    # answer; the oracle must NOT produce it.
    Wm = (W * r["mask"]).astype(np.float32)
    gam_c, scale_c, _ = oracle.absmean_scale(Wm)
    assert gam_c == np.float32(g["control_gamma"][0])
    control = oracle.ternarize(Wm, scale_c)
    assert control.tolist() == [[int(v) for v in g["control_weff"]]]
    assert control.tolist() != weff.tolist()


def test_order_matters_on_gaussian():
    # With gamma fixed, mask(.)Q(w) == Q(mask(.)w); only gamma differs.  For Gaussian W the
    # masked-subset mean is ~0.7446 of the dense mean and ~1.4 % of W_eff entries change.
    W = inputs.latent_weights(512, 1024, seed=11)
    r = oracle.quantize_mask_pack(W)
    weff, mask = oracle.unpack24(r["vals"], r["meta"])
    assert np.array_equal(oracle.ternarize((W * mask).astype(np.float32), r["scale"]), weff)
    Wm = (W * mask).astype(np.float32)
    gm, sm, _ = oracle.absmean_scale(Wm)
    # E|w| over the two largest of four iid half-normals, halved by the mask: closed form is
    # awkward, so only a bracket is asserted here; the ratio is far from 1 either way.
    assert 0.72 < gm / r["scale"] < 0.77
    control = oracle.ternarize(Wm, sm)
    frac = np.mean(control != weff)
    assert 0.008 < frac < 0.02


# ------------------------------------------------------------------------------------------------
# Eq. 1 scale: closed forms.
# ------------------------------------------------------------------------------------------------
def test_gamma_closed_forms():
    # |W| == c (power of two) -> gamma == c exactly, all q = sign
    rng = np.random.default_rng(0)
    sign = rng.choice([-1.0, 1.0], size=(32, 64)).astype(np.float32)
    W = sign * np.float32(0.25)
    g, s, _ = oracle.absmean_scale(W)
    assert g == np.float32(0.25) and s == np.float32(0.25)
    assert np.array_equal(oracle.ternarize(W, s), sign.astype(np.int8))
    # W == 0 -> scale is the clamp 1e-5, all q = 0
    Z = np.zeros((8, 16), np.float32)
    g, s, _ = oracle.absmean_scale(Z)
    assert g == 0.0 and s == np.float32(1e-5)
    assert not oracle.ternarize(Z, s).any()
    # tiny weights below the clamp: gamma < 1e-5 but scale = 1e-5
    Tn = np.full((8, 16), 1e-7, np.float32)
    g, s, _ = oracle.absmean_scale(Tn)
    assert s == np.float32(1e-5) and g < s
    # mean of 1..8 in a known arrangement
    A = np.array([[1, -2, 3, -4, 5, -6, 7, -8]], np.float32)
    g, s, _ = oracle.absmean_scale(A)
    assert g == np.float32(4.5)


def test_ternary_inputs_are_a_fixed_point():
    # W = c * t with t ternary and non-zero fraction f: gamma = f*c, |w|/gamma = 1/f >= 1 > 0.5
    rng = np.random.default_rng(1)
    t = rng.choice([-1, 0, 1], size=(64, 128), p=[0.3, 0.4, 0.3]).astype(np.int8)
    W = t.astype(np.float32) * np.float32(0.037)
    _, s, _ = oracle.absmean_scale(W)
    assert np.array_equal(oracle.ternarize(W, s), t)


def test_ternarize_matches_numpy_rint_division():
    # special case that reduces to library routines: fp32 division, rint (half-even), clip
    W = inputs.latent_weights(128, 256, seed=2)
    _, s, _ = oracle.absmean_scale(W)
    ref = np.clip(np.rint(W / np.float32(s)), -1, 1).astype(np.int8)
    assert np.array_equal(oracle.ternarize(W, s), ref)
    # exact halves: 0.5 -> 0, 1.5 -> 2 -> clamp 1, -0.5 -> 0, 2.5 -> 1
    H = np.array([[0.5, -0.5, 1.5, -1.5, 2.5, 0.49999997, 0.50000006, -0.50000006]], np.float32)
    assert oracle.ternarize(H, 1.0).tolist() == [[0, 0, 1, -1, 1, 0, 1, -1]]


def test_scale_uses_max_not_sum_for_epsilon():
    # gamma + 1e-5 and max(gamma, 1e-5) disagree visibly when gamma ~ 1e-5
    W = np.full((4, 8), 1.6e-5, np.float32)
    _, s, _ = oracle.absmean_scale(W)
    assert s == np.float32(1.6e-5)
    assert (oracle.ternarize(W, s) == 1).all()


def test_power_of_two_and_sign_invariance():
    W = inputs.latent_weights(64, 256, seed=3)
    r = oracle.quantize_mask_pack(W)
    for j in (-3, 5):
        r2 = oracle.quantize_mask_pack((W * np.float32(2.0 ** j)).astype(np.float32))
        assert np.array_equal(r2["vals"], r["vals"]) and np.array_equal(r2["meta"], r["meta"])
        assert r2["scale"] == np.float32(r["scale"] * np.float32(2.0 ** j))
    rn = oracle.quantize_mask_pack(-W)
    assert np.array_equal(rn["vals"], -r["vals"]) and np.array_equal(rn["meta"], r["meta"])


# ------------------------------------------------------------------------------------------------
# Eq. 2 mask: invariants and brute force.
# ------------------------------------------------------------------------------------------------
LEGAL_NIBBLES = {4, 8, 12, 9, 13, 14}


def _brute_mask(W, n_keep, m_group):
    N, K = W.shape
    out = np.zeros((N, K), np.uint8)
    for n in range(N):
        for g in range(K // m_group):
            a = [abs(float(W[n, g * m_group + j])) for j in range(m_group)]
            order = sorted(range(m_group), key=lambda j: (-a[j], j))
            for j in order[:n_keep]:
                out[n, g * m_group + j] = 1
    return out


@pytest.mark.parametrize("n_keep,m_group", [(2, 4), (6, 8), (1, 4), (4, 8)])
def test_mask_brute_force_and_invariants(n_keep, m_group):
    rng = np.random.default_rng(4)
    W = rng.standard_normal((16, 64)).astype(np.float32)
    # inject ties, zeros and sign-mirrored duplicates
    W[0, :8] = 0.0
    W[1, :8] = [1, -1, 1, -1, 2, 2, -2, 2]
    W[2, :8] = [0.5, 0.25, 0.5, 0.25, 0, 0, 1, 0]
    mask = oracle.nm_mask(W, n_keep, m_group)
    assert np.array_equal(mask, _brute_mask(W, n_keep, m_group))
    grp = mask.reshape(16, -1, m_group)
    assert (grp.sum(-1) == n_keep).all()
    a = np.abs(W).reshape(16, -1, m_group)
    kept_min = np.where(grp == 1, a, np.inf).min(-1)
    drop_max = np.where(grp == 0, a, -np.inf).max(-1)
    assert (kept_min >= drop_max).all()


def test_mask_ties_keep_lower_columns():
    W = np.zeros((1, 8), np.float32)
    W[0, 4:] = 3.0
    assert oracle.nm_mask(W).tolist() == [[1, 1, 0, 0, 1, 1, 0, 0]]


def test_mask_comes_from_master_weights_not_from_ternary():
    # group whose ternary image is all ones: only the fp32 magnitudes can rank it
    W = np.array([[0.9, 1.3, 1.1, 1.2, 5, 5, 5, 5]], np.float32)
    mask = oracle.nm_mask(W)
    assert mask[0, :4].tolist() == [0, 1, 0, 1]


def test_pack_layout_and_roundtrip():
    W = inputs.latent_weights(32, 128, seed=5)
    r = oracle.quantize_mask_pack(W)
    assert set(np.unique(r["vals"]).tolist()) <= {-1, 0, 1}
    nibs = np.concatenate([(r["meta"] & 15).ravel(), (r["meta"] >> 4).ravel()])
    assert set(np.unique(nibs).tolist()) <= LEGAL_NIBBLES
    weff, mask = oracle.unpack24(r["vals"], r["meta"])
    assert np.array_equal(mask, r["mask"])
    assert np.array_equal(weff, r["dense_q"] * r["mask"].astype(np.int8))
    # explicit layout on one group: columns 1 and 3 kept -> nibble 1 | 3<<2 = 13
    q = np.array([[0, 1, 0, -1, 1, 0, 0, 1]], np.int8)
    m = np.array([[0, 1, 0, 1, 1, 0, 0, 1]], np.uint8)
    vals, meta = oracle.pack24(q, m)
    assert vals.tolist() == [[1, -1, 1, 1]]
    assert meta.tolist() == [[13 | (12 << 4)]]
    with pytest.raises(ValueError):
        oracle.pack24(q, np.array([[1, 1, 1, 0, 1, 0, 0, 1]], np.uint8))


def test_gaussian_closed_forms(golden_dir):
    g = _read_golden(os.path.join(golden_dir, "gaussian_closed_forms.txt"))
    sigma = 0.02
    N, K = 1024, 2048
    W = inputs.latent_weights(N, K, seed=6, sigma=sigma)
    r = oracle.quantize_mask_pack(W)
    tol = 4.0 / math.sqrt(N * K)
    assert abs(r["scale"] / sigma - g["gamma_over_sigma"][0]) < 2e-3
    assert abs(np.mean(r["dense_q"] == 0) - g["p_zero"][0]) < tol * 2
    assert abs(np.mean(r["vals"] == 0) - g["kept_zero_fraction"][0]) < tol * 2
    weff, _ = oracle.unpack24(r["vals"], r["meta"])
    assert abs(np.mean(weff != 0) - g["weff_density"][0]) < tol * 2


# ------------------------------------------------------------------------------------------------
# Activation quantiser: closed forms.
# ------------------------------------------------------------------------------------------------
def _bf16(a):
    return inputs.f32_to_bf16_bits(np.asarray(a, np.float32))


def test_quant_act_integer_rows_are_identity():
    rng = np.random.default_rng(7)
    x = rng.integers(-127, 128, size=(16, 64)).astype(np.float32)
    x[:, 0] = 127.0 * rng.choice([-1, 1], size=16)
    xq, s = oracle.quant_act(_bf16(x))
    assert np.array_equal(xq, x.astype(np.int8))
    assert (s == np.float32(1.0)).all()


def test_quant_act_half_to_even_and_zero_row():
    x = np.zeros((3, 8), np.float32)
    x[0] = [127, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5]
    x[2] = [-127, 126.5, 125.5, 0, 0, 0, 0, 0]
    xq, s = oracle.quant_act(_bf16(x))
    assert xq[0].tolist() == [127, 0, 2, 2, 0, -2, -2, 4]
    assert not xq[1].any() and s[1] == np.float32(np.float32(1e-5) / np.float32(127.0))
    assert xq[2].tolist()[:3] == [-127, 126, 126]   # 126.5 -> 126 (even); 125.5 -> 126 (bf16: 125.5 exact)


def test_quant_act_properties():
    x = inputs.activations_bf16(64, 512, seed=8)
    xq, s = oracle.quant_act(x)
    xf = inputs.bf16_bits_to_f32(x)
    am = np.abs(xf).argmax(1)
    assert (np.abs(xq[np.arange(64), am].astype(np.int32)) == 127).all()
    assert xq.min() >= -127 and xq.max() <= 127
    assert np.array_equal(s, (np.abs(xf).max(1) / np.float32(127.0)).astype(np.float32))
    # scaling by a power of two leaves the codes unchanged and scales a_scale exactly
    xq2, s2 = oracle.quant_act(_bf16(xf * np.float32(8.0)))
    assert np.array_equal(xq2, xq) and np.array_equal(s2, s * np.float32(8.0))
    # the multiply-by-s_x form, as numpy does it in fp32
    sx = (np.float32(127.0) / np.maximum(np.abs(xf).max(1, keepdims=True), np.float32(1e-5))).astype(np.float32)
    ref = np.clip(np.rint(xf * sx), -128, 127).astype(np.int8)
    assert np.array_equal(xq, ref)


# ------------------------------------------------------------------------------------------------
# Eq. 4: integer accumulation and scaling.
# ------------------------------------------------------------------------------------------------
def test_acc_brute_force_tiny():
    rng = np.random.default_rng(9)
    T, N, K = 5, 6, 16
    xq = rng.integers(-127, 128, size=(T, K)).astype(np.int8)
    W = rng.standard_normal((N, K)).astype(np.float32)
    r = oracle.quantize_mask_pack(W)
    weff, _ = oracle.unpack24(r["vals"], r["meta"])
    brute = [[sum(int(xq[t, k]) * int(weff[n, k]) for k in range(K)) for n in range(N)] for t in range(T)]
    assert oracle.acc_packed(xq, r["vals"], r["meta"]).tolist() == brute
    assert oracle.acc_dense(xq, weff).tolist() == brute
    brute_d = [[sum(int(xq[t, k]) * int(r["dense_q"][n, k]) for k in range(K)) for n in range(N)] for t in range(T)]
    assert oracle.acc_dense(xq, r["dense_q"]).tolist() == brute_d


def test_acc_routes_agree_with_int64_matmul():
    W = inputs.latent_weights(96, 256, seed=10)
    x = inputs.activations_bf16(40, 256, seed=11)
    r = oracle.quantize_mask_pack(W)
    xq, s = oracle.quant_act(x)
    weff, mask = oracle.unpack24(r["vals"], r["meta"])
    ref = xq.astype(np.int64) @ weff.astype(np.int64).T
    a1 = oracle.acc_dense(xq, weff)
    a2 = oracle.acc_packed(xq, r["vals"], r["meta"])
    assert np.array_equal(a1, ref) and np.array_equal(a2, ref)
    assert np.abs(ref).max() <= 127 * 256 // 2
    # dense minus sparse is exactly the pruned part
    ad = oracle.acc_dense(xq, r["dense_q"])
    pruned = xq.astype(np.int64) @ (r["dense_q"].astype(np.int64) * (1 - mask.astype(np.int64))).T
    assert np.array_equal(ad - a1, pruned)
    # sampled variants agree with the full ones
    t_idx, n_idx = inputs.sample_positions(40, 96, 50, seed=1)
    assert np.array_equal(oracle.acc_packed_sampled(xq, r["vals"], r["meta"], t_idx, n_idx), ref[t_idx, n_idx])
    assert np.array_equal(oracle.acc_dense_sampled(xq, r["dense_q"], t_idx, n_idx), ad[t_idx, n_idx])


def test_exact_integer_layer():
    # integer activations (s_x = 1) and ternary weights (fixed point): no quantisation error at
    # all, so y equals gamma * (X @ (W (.) mask)^T) with an exact integer product
    rng = np.random.default_rng(12)
    T, N, K = 8, 16, 64
    X = rng.integers(-127, 128, size=(T, K)).astype(np.float32)
    X[:, 0] = 127
    tern = rng.choice([-1, 0, 1], size=(N, K)).astype(np.int8)
    tern[0, :4] = [1, 1, 1, 1]     # forces a pruning decision among equal magnitudes
    c = np.float32(0.5)
    W = tern.astype(np.float32) * c
    r = oracle.quantize_mask_pack(W)
    xq, s = oracle.quant_act(_bf16(X))
    y, acc = oracle.sparse_bitlinear(xq, s, r["vals"], r["meta"], r["scale"])
    mask = oracle.nm_mask(W)
    ref = X.astype(np.int64) @ (tern.astype(np.int64) * mask).T
    assert np.array_equal(acc, ref)
    assert np.allclose(y, np.float64(r["scale"]) * ref, rtol=1e-6)


def test_dequant_association_and_bias():
    acc = np.array([[3, -5], [70000, 1]], np.int32)
    a_scale = np.array([0.5, 0.25], np.float32)
    y = oracle.dequant(acc, 2.0, a_scale)
    assert y.tolist() == [[3.0, -5.0], [35000.0, 0.5]]
    yb = oracle.dequant(acc, 2.0, a_scale, np.array([1.0, -1.0], np.float32))
    assert yb.tolist() == [[4.0, -6.0], [35001.0, -0.5]]
    # generic scales: float(acc) * fl(scale * a_scale), each product rounded once
    rng = np.random.default_rng(13)
    acc = rng.integers(-300000, 300000, size=(7, 9)).astype(np.int32)
    a_scale = rng.random(7).astype(np.float32)
    sc = np.float32(0.0159)
    s = (sc * a_scale).astype(np.float32)
    ref = (acc.astype(np.float32) * s[:, None]).astype(np.float32)
    assert np.array_equal(oracle.dequant(acc, sc, a_scale), ref)
    rel = np.abs(ref.astype(np.float64) / (np.float64(sc) * a_scale.astype(np.float64))[:, None] - acc)
    assert (rel <= 2 * np.abs(acc) * 2.0 ** -23 + 1e-9).all()


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(14)
    y = rng.standard_normal(4096).astype(np.float32) * np.float32(37.0)
    y[:4] = [1.00390625, 1.01171875, -1.00390625, 3.0]    # exact halves between bf16 neighbours
    ref = torch.from_numpy(y).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.f32_to_bf16_bits(y), ref)
    assert np.array_equal(inputs.f32_to_bf16_bits(y), ref)


# ------------------------------------------------------------------------------------------------
# Flip rate.
# ------------------------------------------------------------------------------------------------
def test_flip_count_cases():
    W = inputs.latent_weights(64, 256, seed=15)
    m0 = oracle.nm_mask(W)
    assert oracle.flip_count(m0, m0) == 0
    # swap the 2nd and 3rd magnitudes of one group -> exactly two positions change
    W2 = W.copy()
    grp = np.abs(W2[3, 8:12])
    order = np.argsort(-grp)
    j2, j3 = 8 + order[1], 8 + order[2]
    W2[3, j2], W2[3, j3] = W2[3, j3], W2[3, j2]
    m1 = oracle.nm_mask(W2)
    assert oracle.flip_count(m0, m1) == 2
    # per group the count is 0, 2 or 4
    Wp = inputs.perturb_weights(W, seed=16, sigma=5e-3)
    mp = oracle.nm_mask(Wp)
    per_group = (m0 != mp).reshape(64, -1, 4).sum(-1)
    assert set(np.unique(per_group).tolist()) <= {0, 2, 4}
    assert oracle.flip_count(m0, mp) == int(per_group.sum())


def test_flip_rate_of_the_dynamic_mask_workload():
    # W ~ N(0, 0.02), one step W += N(0, 1e-4): the flip rate of the 2:4 mask is a few 1e-3
    W = inputs.latent_weights(1024, 2560, seed=17)
    Wp = inputs.perturb_weights(W, seed=18, sigma=1e-4)
    r = oracle.flip_count(oracle.nm_mask(W), oracle.nm_mask(Wp)) / W.size
    assert 2.5e-3 < r < 4.5e-3


# ------------------------------------------------------------------------------------------------
# Algorithm 1: x~ = Q_a(Norm(x)), Norm read as RMSNorm with gain g.
# ------------------------------------------------------------------------------------------------
def _bf16_bits(a):
    return inputs.f32_to_bf16_bits(np.asarray(a, np.float32))


def _bits_to_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def test_norm_quant_act_reduces_to_quant_act_on_unit_rms_rows():
    # rows of +-1 have mean square exactly 1: with eps = 0 and no gain Norm is the identity, and the
    # result must be the (separately pinned) activation quantiser's, bit for bit
    rng = np.random.default_rng(21)
    x = _bf16_bits(rng.choice(np.array([-1.0, 1.0], np.float32), size=(7, 384)))
    r = oracle.norm_quant_act(x, None, 0.0)
    xq, s = oracle.quant_act(x)
    assert np.array_equal(r["xq"], xq) and np.array_equal(r["a_scale"], s)
    assert set(np.unique(r["xq"]).tolist()) == {-127, 127}
    assert np.all(r["a_scale"] == np.float32(1.0) / np.float32(127.0))


def test_norm_quant_act_ignores_power_of_four_scaling():
    # x -> 4x: the mean square is multiplied by 16 exactly, its root by 4 exactly, so with eps = 0 the
    # normalised row -- hence codes and scale -- must not change at all
    x = inputs.activations_bf16(9, 640, seed=22)
    x4 = _bf16_bits(_bits_to_f64(x) * 4.0)
    a = oracle.norm_quant_act(x, None, 0.0, want_xn=True)
    c = oracle.norm_quant_act(x4, None, 0.0, want_xn=True)
    assert np.array_equal(a["xn"], c["xn"])
    assert np.array_equal(a["xq"], c["xq"]) and np.array_equal(a["a_scale"], c["a_scale"])


def test_norm_quant_act_gain():
    x = inputs.activations_bf16(6, 512, seed=23)
    base = oracle.norm_quant_act(x, None, 1e-6)
    half = oracle.norm_quant_act(x, np.full(512, 0.5, np.float32), 1e-6)
    # a power-of-two gain on every channel scales the row exactly: same codes, half the scale
    assert np.array_equal(half["xq"], base["xq"])
    assert np.array_equal(half["a_scale"], base["a_scale"] * np.float32(0.5))
    # a channel with gain 0 quantises to 0; a channel with a dominant gain takes the code +-127
    g = np.ones(512, np.float32)
    g[5] = 0.0
    g[9] = 1000.0
    r = oracle.norm_quant_act(x, g, 1e-6)
    assert np.all(r["xq"][:, 5] == 0)
    assert np.all(np.abs(r["xq"][:, 9].astype(np.int32)) == 127)


def test_norm_quant_act_against_float64():
    T, K = 11, 768
    x = inputs.activations_bf16(T, K, seed=24, token_lognormal_sigma=0.5)
    g = (1.0 + 0.1 * np.random.default_rng(25).standard_normal(K)).astype(np.float32)
    eps = 1e-5
    r = oracle.norm_quant_act(x, g, eps, want_xn=True)
    xf = _bits_to_f64(x)
    xn = xf / np.sqrt((xf ** 2).mean(axis=1, keepdims=True) + eps) * g.astype(np.float64)
    assert np.max(np.abs(r["xn"] - xn) / np.maximum(np.abs(xn), 1e-30)) < 4e-7      # three fp32 roundings
    d = np.maximum(np.abs(xn).max(axis=1, keepdims=True), 1e-5)
    p = xn * (127.0 / d)
    code = np.clip(np.rint(p), -128, 127)
    safe = np.abs(np.abs(p - np.floor(p)) - 0.5) > 1e-3          # away from a rounding boundary
    assert safe.mean() > 0.99
    assert np.array_equal(r["xq"][safe], code[safe].astype(np.int8))
    assert np.max(np.abs(r["xq"].astype(np.float64) - code)) <= 1
    assert np.allclose(r["a_scale"], (d / 127.0).ravel(), rtol=1e-6)
    assert not r["near_tie"].any()


def test_norm_quant_act_degenerate_rows():
    x = np.zeros((3, 256), np.uint16)                              # all-zero rows: eps keeps r finite
    r = oracle.norm_quant_act(x, None, 1e-6)
    assert not r["xq"].any()
    assert np.all(r["a_scale"] == np.float32(1e-5) / np.float32(127.0))
    # constant-magnitude rows: |xn| = 1 (to rounding) whatever the magnitude, so every code is +-127
    for c in (3.0, 0.0078125, 1000.0):
        row = _bf16_bits(np.tile(np.array([c, -c], np.float32), 128))[None, :]
        r = oracle.norm_quant_act(row, None, 0.0, want_xn=True)
        assert np.all(np.abs(r["xq"].astype(np.int32)) == 127)
        assert np.all(np.sign(r["xq"][0, ::2]) == 1) and np.all(np.sign(r["xq"][0, 1::2]) == -1)
        assert abs(float(r["a_scale"][0]) * 127.0 - 1.0) < 3e-7


# ---- general N:M composition (Sec. 2.2; the 6:8 pattern of the main results) -------------------
def test_nm_composition_at_2_of_4_equals_the_packed_route():
    # two routes to W_eff that share no packing code: element-wise composition vs unpacking the
    # compressed values + metadata
    W = inputs.latent_weights(64, 256, seed=71)
    r = oracle.quantize_mask_pack(W)
    w_eff_packed, mask_packed = oracle.unpack24(r["vals"], r["meta"])
    c = oracle.quantize_mask_nm(W, 2, 4)
    assert c["scale"] == r["scale"]
    assert np.array_equal(c["mask"], mask_packed)
    assert np.array_equal(c["w_eff"], w_eff_packed)


def test_nm_composition_6_of_8_hand_case():
    # gamma = mean|W| = (1+2+3+4+5+6+0.5+0.25)/8 = 2.71875; W/gamma rounds to
    # 0 (0.37), 1 (0.74), -1, 1, 1 (1.84 clamps), -1, 0, 0; the two smallest |w| (columns 6, 7) are dropped
    W = np.array([[1.0, 2.0, -3.0, 4.0, 5.0, -6.0, 0.5, -0.25]], np.float32)
    c = oracle.quantize_mask_nm(W, 6, 8)
    assert c["scale"] == np.float32(2.71875)
    assert c["mask"].tolist() == [[1, 1, 1, 1, 1, 1, 0, 0]]
    assert c["w_eff"].tolist() == [[0, 1, -1, 1, 1, -1, 0, 0]]
    # all equal magnitudes: the lower columns win the ties
    c = oracle.quantize_mask_nm(np.full((1, 8), -1.0, np.float32), 6, 8)
    assert c["mask"].tolist() == [[1, 1, 1, 1, 1, 1, 0, 0]]
    assert c["w_eff"].tolist() == [[-1, -1, -1, -1, -1, -1, 0, 0]]


def test_nm_composition_6_of_8_properties_and_negative_control():
    W = inputs.latent_weights(32, 512, seed=72)
    c = oracle.quantize_mask_nm(W, 6, 8)
    grp_mask = c["mask"].reshape(32, -1, 8)
    assert (grp_mask.sum(-1) == 6).all()
    a = np.abs(W).reshape(32, -1, 8)
    kept_min = np.where(grp_mask == 1, a, np.inf).min(-1)
    drop_max = np.where(grp_mask == 0, a, -np.inf).max(-1)
    assert (kept_min >= drop_max).all()
    # gamma is the DENSE mean (quant-then-mask, Eq. 3): same scale as the 2:4 and the unmasked paths
    assert c["scale"] == oracle.quantize_mask_nm(W, 2, 4)["scale"] == oracle.quantize_mask_nm(W, 8, 8)["scale"]
    # 8:8 is the dense BitLinear weight
    assert np.array_equal(oracle.quantize_mask_nm(W, 8, 8)["w_eff"], oracle.ternarize(W, c["scale"]))
    # negative control: gamma from the masked subset (mask-then-quant) gives another matrix
    Wm = W * c["mask"]
    _, scale_m, _ = oracle.absmean_scale(Wm)
    assert scale_m != c["scale"]
    assert not np.array_equal(oracle.ternarize(Wm, scale_m), c["w_eff"])


def test_nm_bitlinear_is_the_integer_matmul():
    rng = np.random.default_rng(73)
    W = inputs.latent_weights(16, 64, seed=73)
    c = oracle.quantize_mask_nm(W, 6, 8)
    xq = rng.integers(-128, 128, size=(5, 64), dtype=np.int8)
    a_scale = rng.uniform(0.01, 0.1, size=5).astype(np.float32)
    y, acc = oracle.nm_bitlinear(xq, a_scale, c["w_eff"], c["scale"])
    ref = xq.astype(np.int64) @ c["w_eff"].astype(np.int64).T
    assert np.array_equal(acc, ref)
    s = np.float32(c["scale"]) * a_scale
    assert np.array_equal(y, (ref.astype(np.float32).T * s).T.astype(np.float32))


# ---- packed storage of the kept values (2 bits each) ------------------------------------------------
def test_pack_vals2_hand_case_and_all_states():
    # all nine (v0, v1) states in one row, padded to a legal width with (0, 0) groups
    states = [(v0, v1) for v0 in (-1, 0, 1) for v1 in (-1, 0, 1)]
    G = 16
    vals = np.zeros((1, 2 * G), np.int8)
    for g, (v0, v1) in enumerate(states):
        vals[0, 2 * g], vals[0, 2 * g + 1] = v0, v1
    out = oracle.pack_vals2(vals)
    assert out.shape == (1, G // 2)
    nibs = [(v0 + 1) | ((v1 + 1) << 2) for v0, v1 in states] + [5] * (G - 9)     # (0,0) -> 1 | 1 << 2 = 5
    expect = [nibs[2 * b] | (nibs[2 * b + 1] << 4) for b in range(G // 2)]
    assert out[0].tolist() == expect
    assert out[0, 0] == (0 | (0 << 2)) | ((0 | (1 << 2)) << 4)       # (-1,-1) then (-1,0): 0x40
    assert np.array_equal(oracle.unpack_vals2(out), vals)


def test_pack_vals2_round_trip_and_rejections():
    W = inputs.latent_weights(64, 512, seed=91)
    r = oracle.quantize_mask_pack(W)
    v2 = oracle.pack_vals2(r["vals"])
    assert (v2.size + r["meta"].size) * 8 == 2 * W.size              # 2 bits per weight with the metadata
    assert np.array_equal(oracle.unpack_vals2(v2), r["vals"])
    bad = r["vals"].copy()
    bad[0, 0] = 2
    with pytest.raises(ValueError):
        oracle.pack_vals2(bad)
    badb = v2.copy()
    badb[0, 0] |= 3
    with pytest.raises(ValueError):
        oracle.unpack_vals2(badb)


# ------------------------------------------------------------------------------------------------
# backward under the dual straight-through estimator (Sec. 2.3, Eq. 5; Algorithm 2's backward)
# ------------------------------------------------------------------------------------------------
def _tiny_backward_case(seed, T=5, N=4, K=8):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    x = inputs.f32_to_bf16_bits(rng.standard_normal((T, K)).astype(np.float32))
    dy = inputs.f32_to_bf16_bits(rng.standard_normal((T, N)).astype(np.float32))
    scale = oracle.absmean_scale(W)[1]
    mask = oracle.nm_mask(W)
    w_eff = oracle.apply_mask(oracle.ternarize(W, scale), mask)
    xq, a_scale = oracle.quant_act(x)
    return W, mask, w_eff, np.float32(scale), xq, a_scale, dy


def test_backward_is_brute_force_on_tiny_inputs():
    # pure-Python triple loops over the definition, operand roundings written out by hand
    W, mask, w_eff, scale, xq, a_scale, dy = _tiny_backward_case(1)
    T, K = xq.shape
    N = w_eff.shape[0]
    dY = inputs.bf16_bits_to_f32(dy).astype(np.float64)
    s_b = float(inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(np.array([scale], np.float32)))[0])
    dW = np.zeros((N, K)); dX = np.zeros((T, K))
    for t in range(T):
        for k in range(K):
            xq_b = float(inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(np.array([np.float32(xq[t, k]) * a_scale[t]], np.float32)))[0])
            for n in range(N):
                dW[n, k] += dY[t, n] * xq_b
                dX[t, k] += dY[t, n] * (float(w_eff[n, k]) * s_b)
    gx, gw = oracle.backward_dual_ste(dy, xq, a_scale, w_eff, scale)
    assert np.allclose(gw, dW, rtol=1e-13, atol=1e-15)
    assert np.allclose(gx, dX, rtol=1e-13, atol=1e-15)


def test_backward_matches_finite_differences_of_the_linear_map():
    # y = x_q w_masked^T is bilinear, so central differences of L = sum(G * y) in one entry of
    # w_masked (or of x_q) give the gradients exactly: a transposed operand or a wrong index fails
    W, mask, w_eff, scale, xq, a_scale, dy = _tiny_backward_case(2, T=6, N=3, K=8)
    G = inputs.bf16_bits_to_f32(dy).astype(np.float64)
    xq_b = oracle.fake_quant_act_bf16(xq, a_scale)
    w_b = w_eff.astype(np.float64) * float(oracle.bf16_round(np.array([scale], np.float32))[0])
    loss = lambda xa, wa: float(np.sum(G * np.einsum("tk,nk->tn", xa, wa)))
    gx, gw = oracle.backward_dual_ste(dy, xq, a_scale, w_eff, scale)
    h = 0.5
    for (n, k) in [(0, 0), (2, 7), (1, 3)]:
        wp, wm = w_b.copy(), w_b.copy()
        wp[n, k] += h; wm[n, k] -= h
        assert abs((loss(xq_b, wp) - loss(xq_b, wm)) / (2 * h) - gw[n, k]) <= 1e-9 * max(1.0, abs(gw[n, k]))
    for (t, k) in [(0, 0), (5, 7), (3, 2)]:
        xp, xm = xq_b.copy(), xq_b.copy()
        xp[t, k] += h; xm[t, k] -= h
        assert abs((loss(xp, w_b) - loss(xm, w_b)) / (2 * h) - gx[t, k]) <= 1e-9 * max(1.0, abs(gx[t, k]))


def test_backward_adjoint_identities():
    # <dY, forward(x_q, w)> = <dX, x_q> = <dW, w>: the backward maps are the adjoints of the forward one
    W, mask, w_eff, scale, xq, a_scale, dy = _tiny_backward_case(3, T=7, N=8, K=16)
    G = inputs.bf16_bits_to_f32(dy).astype(np.float64)
    xq_b = oracle.fake_quant_act_bf16(xq, a_scale)
    w_b = w_eff.astype(np.float64) * float(oracle.bf16_round(np.array([scale], np.float32))[0])
    gx, gw = oracle.backward_dual_ste(dy, xq, a_scale, w_eff, scale)
    lhs = float(np.sum(G * (xq_b @ w_b.T)))
    assert abs(lhs - float(np.sum(gx * xq_b))) <= 1e-12 * max(1.0, abs(lhs))
    assert abs(lhs - float(np.sum(gw * w_b))) <= 1e-12 * max(1.0, abs(lhs))


def test_backward_one_hot_gradient_reads_rows_back():
    W, mask, w_eff, scale, xq, a_scale, dy = _tiny_backward_case(4, T=4, N=4, K=8)
    one = np.zeros((4, 4), np.float32)
    one[2, 1] = 1.0                                           # dL/dy[t=2][n=1] = 1
    gx, gw = oracle.backward_dual_ste(inputs.f32_to_bf16_bits(one), xq, a_scale, w_eff, scale)
    xq_b = oracle.fake_quant_act_bf16(xq, a_scale)
    s_b = float(oracle.bf16_round(np.array([scale], np.float32))[0])
    assert np.array_equal(gw[1], xq_b[2]) and not gw[[0, 2, 3]].any()
    assert np.array_equal(gx[2], w_eff[1].astype(np.float64) * s_b) and not gx[[0, 1, 3]].any()


def test_backward_weight_gradient_is_dense_not_gated_by_the_mask():
    # Eq. 5: the mask is transparent, pruned weights receive their gradient; the gated alternative
    # (M (.) dW) is the negative control and must differ
    W, mask, w_eff, scale, xq, a_scale, dy = _tiny_backward_case(5, T=9, N=8, K=16)
    gw = oracle.backward_dw(dy, xq, a_scale)
    pruned = mask == 0
    assert pruned.sum() == mask.size // 2
    assert np.count_nonzero(gw[pruned]) > 0.9 * pruned.sum()
    assert not np.array_equal(gw, gw * mask)


def test_backward_operand_roundings():
    # the saved activations are held in bf16: integer codes times a power-of-two scale are exact,
    # a scale with a long mantissa is rounded once (ties to even)
    xq = np.array([[127, -3, 64, 1]], np.int8)
    assert np.array_equal(oracle.fake_quant_act_bf16(xq, np.array([0.25], np.float32)), xq.astype(np.float64) * 0.25)
    s = np.float32(1.0 + 2.0 ** -9)                            # 127 * s needs more than 8 bits
    got = oracle.fake_quant_act_bf16(np.array([[127, 1]], np.int8), np.array([s], np.float32))
    assert got[0, 0] == 127.0 and got[0, 1] == 1.0             # 127.248 -> 127 (8-bit significand), 1.00195 -> 1
    assert oracle.bf16_round(np.array([1.0 + 2.0 ** -8], np.float32))[0] == 1.0          # tie -> even
    assert oracle.bf16_round(np.array([1.0 + 3 * 2.0 ** -8], np.float32))[0] == 1.0 + 2.0 ** -6


def test_near_tie_flag_fires_when_the_summation_order_decides_gamma():
    # gamma is defined with a double-precision sum; the oracle flags a matrix whose gamma depends on
    # the ORDER of that sum so that parity tests skip the seed instead of blaming a kernel.  Built by
    # hand: 2^30 + 64 + 126 x 2^-23.  Added one by one, every 2^-23 is half an ulp of the running sum
    # and is rounded away (ties to even): S = 2^30 + 64, S / 128 = 2^23 + 0.5 exactly, which rounds to
    # the even fp32 neighbour 2^23.  Added pairwise (halves of 64), the second half sums to 2^-17 first
    # and survives: S / 128 = 2^23 + 0.5 + 2^-24 rounds up to 2^23 + 1.
    W = np.full((1, 128), 2.0 ** -23, np.float32)
    W[0, 0] = 2.0 ** 30
    W[0, 1] = 64.0
    gamma, scale, near_tie = oracle.absmean_scale(W)
    assert gamma == np.float32(2.0 ** 23) and scale == gamma
    assert near_tie
    # an ordinary matrix is not flagged
    assert not oracle.absmean_scale(inputs.latent_weights(128, 256, seed=3))[2]
    # a sum that lies ON an fp32 midpoint is flagged even when the two orders the oracle tries agree
    # (without the second half both give 2^30 + 64): a third order could still round the other way
    W[0, 64:] = 0.0
    assert oracle.absmean_scale(W)[2]
    # ... and one that is a comfortable 2^-30 (relative) away from the midpoint is not
    V = np.zeros((1, 128), np.float32)
    V[0, 0] = 2.0 ** 30
    V[0, 1] = 64.0 + 2.0 ** -4
    assert not oracle.absmean_scale(V)[2]
