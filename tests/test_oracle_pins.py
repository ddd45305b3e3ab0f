"""Pins for the CPU oracle: what the paper and the mathematics fix.

Each pin is a function of the oracle module so that the mutation tests at the
end can run the same pins against a copy of the oracle with one planted mistake
and check that some pin catches it.
"""
import itertools
import os
import types

import numpy as np
import pytest

from conftest import GOLDEN, read_golden
from oracle import eqat_oracle as ORACLE
from workloads import LINEARS


def _bf16_exact(x):
    """Round a float array to values representable in bfloat16 (8 significant bits)."""
    u = np.asarray(x, np.float32).view(np.uint32)
    u = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return u.view(np.float32)


def _rand_case(seed, out=6, groups=3, group=8, bits=2, spread=1.0):
    g = np.random.default_rng(seed)
    W = _bf16_exact(g.standard_normal((out, groups * group)) * 0.02)
    s = (np.abs(g.standard_normal((out, groups))) * 0.004 * spread + 0.002).astype(np.float32)
    z = g.integers(0, (1 << bits), size=(out, groups)).astype(np.float32)
    return W, s, z


# --------------------------------------------------------------------------- Eq. 1-5, worked example
def pin_worked_example(o):
    gd = read_golden("ste_one_group_w2.txt")
    bits, group = int(gd["bits"][0]), int(gd["group"][0])
    W = np.array([gd["w"]], np.float32)
    s = np.array([gd["s"]], np.float32)
    z = np.array([gd["z"]], np.float32)
    q, r, p = o.quantize_codes(W, s, z, bits, group)
    assert q.tolist() == [[int(v) for v in gd["code"]]]
    assert r.tolist() == [gd["round"]]
    np.testing.assert_array_equal(o.dequantize(q, s, z, group), [gd["w_hat"]])
    np.testing.assert_array_equal(o.fake_quant_weight(W, s, z, bits, group), [gd["w_hat"]])
    a, b, c = o.ste_partials(W, s, z, bits, group, 0)
    np.testing.assert_array_equal(a, [gd["dwhat_dw"]])
    np.testing.assert_allclose(b, [gd["dwhat_ds"]], rtol=0, atol=1e-12)
    np.testing.assert_array_equal(c, [gd["dwhat_dz"]])
    _, _, c1 = o.ste_partials(W, s, z, bits, group, 1)
    np.testing.assert_array_equal(c1, [gd["dwhat_dz_literal"]])
    G = np.array([gd["G"]])
    dW, ds, dz = o.ste_bwd(G, W, s, z, bits, group, 0)
    np.testing.assert_array_equal(dW, [gd["dW"]])
    np.testing.assert_allclose(ds, [gd["ds"]], atol=1e-12)
    np.testing.assert_allclose(dz, [gd["dz"]], atol=1e-12)
    _, _, dz1 = o.ste_bwd(G, W, s, z, bits, group, 1)
    np.testing.assert_allclose(dz1, [gd["dz_literal"]], atol=1e-12)


def pin_rounding_is_half_to_even(o):
    # w/s = 0.5, 1.5, 2.5, -0.5, -1.5 with s = 1, z = 4, 4 bits (no clamping)
    W = np.array([[0.5, 1.5, 2.5, -0.5, -1.5, 3.5, 0.0, 1.0]], np.float32)
    s = np.ones((1, 1), np.float32)
    z = np.full((1, 1), 4.0, np.float32)
    q, r, _ = o.quantize_codes(W, s, z, 4, 8)
    assert r.tolist() == [[0, 2, 2, -0, -2, 4, 0, 1]]
    assert q.tolist() == [[4, 6, 6, 4, 2, 8, 4, 5]]


def pin_inclusive_bounds(o):
    # pre-clamp value exactly 0 and exactly Q are in range (Eqs. 3-5 print <=)
    W = np.array([[-1.0, 2.0, -2.0, 3.0]], np.float32)       # s=1, z=1, Q=3: p = 0, 3, -1, 4
    s = np.ones((1, 1), np.float32)
    z = np.ones((1, 1), np.float32)
    a, b, c = o.ste_partials(W, s, z, 2, 4, 0)
    assert a.tolist() == [[1, 1, 0, 0]]
    assert b.tolist() == [[0, 0, -1, 2]]
    assert c.tolist() == [[0, 0, -1, -1]]


# --------------------------------------------------------------------------- quantiser invariants
def pin_quantiser_invariants(o):
    for bits in (2, 3, 4):
        Q = (1 << bits) - 1
        W, s, z = _rand_case(10 + bits, bits=bits)
        q, r, p = o.quantize_codes(W, s, z, bits, 8)
        assert q.dtype.kind == "i" and q.min() >= 0 and q.max() <= Q
        assert q.min() == 0 and q.max() == Q          # the case does exercise both clamps
        What = o.fake_quant_weight(W, s, z, bits, 8)
        # on the per-group grid {(k - z) s}
        k = What / np.repeat(s.astype(np.float64), 8, 1) + np.repeat(z.astype(np.float64), 8, 1)
        np.testing.assert_allclose(k, np.rint(k), atol=1e-9)
        assert (np.rint(k) == q).all()
        # idempotence: quantising the dequantised weight gives the same code
        q2, _, _ = o.quantize_codes(What.astype(np.float32), s, z, bits, 8)
        assert (q2 == q).all()
        # s = 1, z = 0 reduces to clamp(rint(w))
        Wi = (np.random.default_rng(5).standard_normal((4, 16)) * 4).astype(np.float32)
        q3, _, _ = o.quantize_codes(Wi, np.ones((4, 2), np.float32), np.zeros((4, 2), np.float32), bits, 8)
        assert (q3 == np.clip(np.rint(Wi), 0, Q)).all()
        # weights already on the grid are reproduced exactly (s a power of two keeps it exact)
        s2 = np.full((4, 2), 0.25, np.float32)
        z2 = np.full((4, 2), 1.0, np.float32)
        codes = np.random.default_rng(6).integers(0, Q + 1, (4, 16))
        Wg = ((codes - 1.0) * 0.25).astype(np.float32)
        np.testing.assert_array_equal(o.fake_quant_weight(Wg, s2, z2, bits, 8), Wg)


def pin_zero_point_is_rounded_in_forward(o):
    W, s, z = _rand_case(3)
    zf = z + np.float32(0.3)
    np.testing.assert_array_equal(o.fake_quant_weight(W, s, zf, 2, 8), o.fake_quant_weight(W, s, z, 2, 8))


# --------------------------------------------------------------------------- STE gradients vs the forward
def pin_ste_against_forward(o):
    """Identities tying Eqs. 3-5 to Eq. 1-2's own output:
    in range: w_hat - w = s * (round(w/s) - w/s); clamped: w_hat = s * d w_hat/d s.
    Clamped elements: w_hat(s + h) - w_hat(s) = h * d w_hat/d s exactly (Eq. 2 is
    linear in s at a fixed code); w_hat(z + 1) - w_hat(z) = d w_hat/d z for
    elements whose branch does not change."""
    for bits in (2, 3, 4):
        Q = (1 << bits) - 1
        W, s, z = _rand_case(20 + bits, out=16, groups=4, bits=bits)
        s64 = np.repeat(s.astype(np.float64), 8, 1)
        What = o.fake_quant_weight(W, s, z, bits, 8)
        a, b, c = o.ste_partials(W, s, z, bits, 8, 0)
        inside = a == 1
        assert inside.any() and (~inside).any()
        np.testing.assert_allclose((What - W.astype(np.float64))[inside], (s64 * b)[inside], atol=1e-9)
        np.testing.assert_allclose(What[~inside], (s64 * b)[~inside], atol=1e-12)
        # finite difference in s on clamped elements far from the clamp threshold
        _, r, p = o.quantize_codes(W, s, z, bits, 8)
        far = (p < -1) | (p > Q + 1)
        assert far.any()
        h = np.float32(2.0 ** -12)
        s_h = (s * (1 + h)).astype(np.float32)
        What_h = o.fake_quant_weight(W, s_h, z, bits, 8)
        _, _, p_h = o.quantize_codes(W, s_h, z, bits, 8)
        still = far & ((p_h < 0) | (p_h > Q))
        ds_el = np.repeat((s_h.astype(np.float64) - s.astype(np.float64)), 8, 1)
        np.testing.assert_allclose((What_h - What)[still], (ds_el * b)[still], rtol=1e-12, atol=1e-15)
        # unit difference in z
        What_z = o.fake_quant_weight(W, s, z + 1, bits, 8)
        a_z, _, _ = o.ste_partials(W, s, z + 1, bits, 8, 0)
        same = (a == a_z)
        np.testing.assert_allclose((What_z - What)[same], c[same], atol=1e-12)
        # literal Eq. 4 differs from the chain-rule form by the factor s
        _, _, c1 = o.ste_partials(W, s, z, bits, 8, 1)
        np.testing.assert_allclose(c1 * s64, c, atol=0)
        # chain rule with group sums
        G = np.random.default_rng(1).standard_normal(W.shape)
        dW, ds, dz = o.ste_bwd(G, W, s, z, bits, 8, 0)
        for oo, gg in itertools.product(range(W.shape[0]), range(s.shape[1])):
            sl = slice(gg * 8, gg * 8 + 8)
            assert abs(ds[oo, gg] - sum(G[oo, j] * b[oo, j] for j in range(sl.start, sl.stop))) < 1e-12
            assert abs(dz[oo, gg] - sum(G[oo, j] * c[oo, j] for j in range(sl.start, sl.stop))) < 1e-12
        np.testing.assert_array_equal(dW, G * a)


# --------------------------------------------------------------------------- contractions
def pin_contractions(o):
    g = np.random.default_rng(7)
    T, out, in_f = 5, 4, 6
    X = g.standard_normal((T, in_f)); Wh = g.standard_normal((out, in_f)); dY = g.standard_normal((T, out))
    Y = o.linear_fwd(X, Wh); dX = o.linear_bwd_dx(dY, Wh); G = o.weight_grad(dY, X)
    assert Y.shape == (T, out) and dX.shape == (T, in_f) and G.shape == (out, in_f)
    for t, oo in itertools.product(range(T), range(out)):
        assert abs(Y[t, oo] - sum(X[t, j] * Wh[oo, j] for j in range(in_f))) < 1e-12
    for t, j in itertools.product(range(T), range(in_f)):
        assert abs(dX[t, j] - sum(dY[t, oo] * Wh[oo, j] for oo in range(out))) < 1e-12
    for oo, j in itertools.product(range(out), range(in_f)):
        assert abs(G[oo, j] - sum(dY[t, oo] * X[t, j] for t in range(T))) < 1e-12
    # adjoint identities <dY, Y> = <dX, X> = <G, W_hat>
    a = (dY * Y).sum(); b = (dX * X).sum(); c = (G * Wh).sum()
    assert abs(a - b) < 1e-10 and abs(a - c) < 1e-10
    # one-hot X picks out a column of W_hat
    E = np.eye(in_f)
    np.testing.assert_array_equal(o.linear_fwd(E, Wh), Wh.T)


# --------------------------------------------------------------------------- E2E-QP gradients
def pin_e2e_ds(o):
    g = np.random.default_rng(11)
    T, out, groups, group, bits = 7, 5, 3, 4, 2
    in_f = groups * group
    X = g.standard_normal((T, in_f)); dY = g.standard_normal((T, out))
    q = g.integers(0, 4, (out, in_f)); z = g.integers(0, 4, (out, groups)).astype(np.float32)
    s = (np.abs(g.standard_normal((out, groups))) + 0.1)
    ds = o.e2e_ds(dY, X, q, z, group)
    # brute force
    for oo, gg in itertools.product(range(out), range(groups)):
        acc = 0.0
        for j in range(gg * group, (gg + 1) * group):
            gij = sum(dY[t, oo] * X[t, j] for t in range(T))
            acc += gij * (q[oo, j] - z[oo, gg])
        assert abs(ds[oo, gg] - acc) < 1e-12
    # Y is linear in s: a unit step in one s changes <dY, Y> by exactly ds
    def loss(s_):
        return (dY * o.linear_fwd(X, o.dequantize(q, s_, z, group))).sum()
    L0 = loss(s)
    for oo, gg in itertools.product(range(out), range(groups)):
        s1 = s.copy(); s1[oo, gg] += 1.0
        assert abs((loss(s1) - L0) - ds[oo, gg]) < 1e-9
    # Euler: sum s * ds = <dY, Y>
    assert abs((s * ds).sum() - L0) < 1e-9
    # zero-point gradient: unit step in z (integers) changes the loss by dz exactly
    dz = o.e2e_dz(dY, X, s, group)
    for oo, gg in itertools.product(range(out), range(groups)):
        z1 = z.copy(); z1[oo, gg] += 1.0
        L1 = (dY * o.linear_fwd(X, o.dequantize(q, s, z1, group))).sum()
        assert abs((L1 - L0) - dz[oo, gg]) < 1e-9


# --------------------------------------------------------------------------- min/max initialisation
def pin_real_zero_point(o):
    """E2E-QP with a trained, real-valued zero point: Eq. 2 uses it unrounded.  Eq. 2 is linear in z, so
    W_hat(z) = W_hat(0) - z s exactly (up to the product's rounding), finite differences in z are exact for any
    step, and an integer-valued z gives the frozen-zero-point result bit for bit."""
    g = np.random.default_rng(21)
    q = g.integers(0, 4, (5, 24))
    s = (np.abs(g.standard_normal((5, 3))) * 0.01 + 0.002).astype(np.float32)
    z = (g.random((5, 3)) * 3).astype(np.float32)                   # fractional
    s_el, z_el = np.repeat(s.astype(np.float64), 8, 1), np.repeat(z.astype(np.float64), 8, 1)
    Wr = o.dequantize(q, s, z, 8, real_zero_point=True)
    np.testing.assert_allclose(Wr, o.dequantize(q, s, np.zeros_like(z), 8) - z_el * s_el, rtol=0, atol=1e-15)
    assert np.abs(Wr - o.dequantize(q, s, z, 8)).max() > 1e-4         # rounding z would be a different layer
    # hand value: q = 3, z = 1.25, s = 0.5  ->  (3 - 1.25) * 0.5 = 0.875
    assert o.dequantize(np.array([[3]]), np.array([[0.5]], np.float32), np.array([[1.25]], np.float32), 1,
                        real_zero_point=True)[0, 0] == 0.875
    zi = np.rint(z)
    np.testing.assert_array_equal(o.dequantize(q, s, zi, 8, real_zero_point=True), o.dequantize(q, s, zi, 8))
    # the gradients: ds is linear in z as well, dz = -s * sum G is the exact derivative of the loss <dY, Y> in z
    X = g.standard_normal((7, 24)); dY = g.standard_normal((7, 5))
    G = o.weight_grad(dY, X)
    ds = o.e2e_ds(dY, X, q, z, 8, real_zero_point=True)
    brute = np.array([[sum(G[r, 8 * k + j] * (q[r, 8 * k + j] - float(z[r, k])) for j in range(8)) for k in range(3)]
                      for r in range(5)])
    np.testing.assert_allclose(ds, brute, rtol=1e-12, atol=1e-12)
    loss = lambda zz: float((dY * o.linear_fwd(X, o.dequantize(q, s, zz, 8, real_zero_point=True))).sum())
    dz = o.e2e_dz(dY, X, s, 8)
    for r, k, h in ((0, 0, 0.37), (4, 2, -1.6)):
        z2 = z.astype(np.float64).copy(); z2[r, k] += h
        assert abs((loss(z2) - loss(z.astype(np.float64))) / h - dz[r, k]) <= 1e-9 * (1 + abs(dz[r, k]))


def pin_minmax(o):
    W = np.array([[-0.3, 0.1, 0.6, 0.0, 1.0, 1.0, 1.0, 1.0]], np.float32)
    s, z = o.minmax_init(W, 2, 4)
    np.testing.assert_allclose(s, [[np.float32(0.9) / np.float32(3), 2.0 ** -14]], rtol=1e-7)
    assert z.tolist() == [[1.0, 0.0]]          # -rint(-0.3/0.3) = 1 ; constant group: -rint(1/2^-14) clamps to 0
    # with min/max initialisation the extremes of each group get codes 0..Q without clamping error
    g = np.random.default_rng(2)
    Wr = _bf16_exact(g.standard_normal((8, 64)) * 0.02)
    for bits in (2, 3, 4):
        s, z = o.minmax_init(Wr, bits, 16)
        assert s.dtype == np.float32 and z.dtype == np.float32
        assert (z == np.rint(z)).all() and z.min() >= 0 and z.max() <= (1 << bits) - 1
        What = o.fake_quant_weight(Wr, s, z, bits, 16)
        err = np.abs(What - Wr).reshape(8, 4, 16).max(axis=2)
        assert (err <= 1.0001 * s).all()       # at most one step (half a step away from the clamps)


# --------------------------------------------------------------------------- codec
def _golden_pack_lines():
    with open(os.path.join(GOLDEN, "pack_bytes.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                b, codes, by = [x.strip() for x in line.split("|")]
                yield int(b), [int(c) for c in codes.split()], [int(x, 16) for x in by.split()]


def pin_pack_golden(o):
    n = 0
    for bits, codes, by in _golden_pack_lines():
        assert o.pack_stream(codes, bits).tolist() == by
        assert o.unpack_stream(np.array(by, np.uint8), bits, len(codes)).tolist() == codes
        n += 1
    assert n >= 5


def pin_pack_roundtrip_and_bigint(o):
    # exhaustive rows: all 4^4 2-bit bytes, all 16^2 4-bit bytes, 4096 sampled + structured 3-bit triples
    for bits, count in ((2, 4), (4, 2)):
        for codes in itertools.product(range(1 << bits), repeat=count):
            p = o.pack_stream(codes, bits)
            assert p.size == 1
            assert int(p[0]) == sum(c << (bits * j) for j, c in enumerate(codes))
            assert tuple(o.unpack_stream(p, bits, count).tolist()) == codes
    g = np.random.default_rng(0)
    cases = [g.integers(0, 8, 8).tolist() for _ in range(4096)]
    cases += [[(i >> (3 * j)) & 7 if j < 4 else 0 for j in range(8)] for i in range(4096)]
    for codes in cases:
        p = o.pack_stream(codes, 3)
        assert p.size == 3
        assert int.from_bytes(bytes(p.tolist()), "little") == sum(c << (3 * j) for j, c in enumerate(codes))
        assert o.unpack_stream(p, 3, 8).tolist() == list(codes)
    for bits in (2, 3, 4):
        q = g.integers(0, 1 << bits, (5, 64))
        P = o.pack_rows(q, bits)
        assert P.shape == (5, 64 * bits // 8) and P.dtype == np.uint8
        assert (o.unpack_rows(P, bits, 64) == q).all()
        for row in range(5):
            assert int.from_bytes(bytes(P[row].tolist()), "little") == sum(int(c) << (bits * j) for j, c in enumerate(q[row]))


def pin_sizes(o):
    """bits/param = N + (N+16)/g and the model sizes the paper prints for Llama-2-7B.
    Block count (32), vocabulary (32000) and hidden size come from the public
    model configuration; the paper keeps embeddings, head and norms in FP16."""
    per_block = sum(l.out_features * l.in_features * l.count for l in LINEARS["7b"])
    assert per_block == 202_375_168                           # Table "ptq_variants": 202.4M weights per block
    assert round(per_block / 1e6, 1) == 202.4
    assert round(2 * per_block / 64 / 1e6, 1) == 6.3          # s and z at g64: 6.3M
    assert round((per_block + 2 * per_block / 64) / 1e6, 1) == 208.7
    total_params = 6_738_415_616
    rest = total_params - 32 * per_block
    assert round(total_params * 2 / 2 ** 30, 2) == 12.55
    with open(os.path.join(GOLDEN, "bits_per_param.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert len(rows) == 9
    for bits, group, bpp, gib in rows:
        bits, group = int(bits), int(group)
        nbytes = sum(o.packed_bytes(l.out_features, l.in_features, bits, group) * l.count for l in LINEARS["7b"])
        got_bpp = 8.0 * nbytes / per_block
        assert abs(got_bpp - (bits + (bits + 16) / group)) < 1e-9
        assert abs(got_bpp - float(bpp)) <= 0.0051
        if bits != 3:      # the printed 3-bit sizes exceed what the printed bits/param give (see the fixture)
            assert abs((32 * nbytes + 2 * rest) / 2 ** 30 - float(gib)) <= 0.0051
    # E2E-QP variant with trainable fp16 zero points: 2 + 32/64 = 2.50 bits (Table "e2e-ft-variants")
    assert 2 + 32 / 64 == 2.5
    # quantize_pack output sizes
    W, s, z = _rand_case(1, out=4, groups=2, group=64)
    P, z8, s16 = o.quantize_pack(W, s, z, 2, 64)
    assert P.shape == (4, 32) and z8.shape == (4, 2) and s16.dtype == np.float16 and z8.dtype == np.uint8
    q, _, _ = o.quantize_codes(W, s, z, 2, 64)
    assert (o.unpack_rows(P, 2, 128) == q).all() and (z8 == z).all()


def pin_handoff_side_outputs(o):
    """Step sizes as FP16 bit patterns and zero points as N-bit bytes, against hand-derived values."""
    rows = []
    with open(os.path.join(GOLDEN, "handoff_side_outputs.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append([x.strip() for x in line.split("|")])
    s_rows = [(float(v), int(h, 16)) for k, v, h in rows if k == "s"]
    assert len(s_rows) == 4
    for kind, bits in (("z2", 2), ("z4", 4)):
        z_rows = [(float(v), int(b)) for k, v, b in rows if k == kind]
        assert len(z_rows) >= 3
        ng = len(z_rows)
        s = np.array([[s_rows[i % len(s_rows)][0] for i in range(ng)]], np.float32)
        z = np.array([[v for v, _ in z_rows]], np.float32)
        W = np.zeros((1, ng * 8), np.float32)
        P, z8, s16 = o.quantize_pack(W, s, z, bits, 8)
        assert z8.dtype == np.uint8 and s16.dtype == np.float16
        assert z8.tolist() == [[b for _, b in z_rows]]
        assert s16.view(np.uint16).tolist() == [[s_rows[i % len(s_rows)][1] for i in range(ng)]]
        # w = 0 quantises to clamp(0 + rint(z), 0, Q): the packed codes repeat the stored zero point
        assert (o.unpack_rows(P, bits, ng * 8) == np.repeat(z8, 8, axis=1)).all()


def pin_shapes_other_models(o):
    assert sum(l.out_features * l.in_features * l.count for l in LINEARS["13b"]) == 317_194_240
    assert sum(l.out_features * l.in_features * l.count for l in LINEARS["70b"]) == 855_638_016
    # shapes of the paper's linear-speed table (out x in)
    shapes = {(l.out_features, l.in_features) for m in LINEARS.values() for l in m}
    for sh in ((4096, 4096), (11008, 4096), (5120, 5120), (13824, 5120), (8192, 8192), (28672, 8192)):
        assert sh in shapes


PINS = [pin_worked_example, pin_rounding_is_half_to_even, pin_inclusive_bounds, pin_quantiser_invariants,
        pin_zero_point_is_rounded_in_forward, pin_ste_against_forward, pin_contractions, pin_e2e_ds,
        pin_real_zero_point, pin_minmax, pin_pack_golden, pin_pack_roundtrip_and_bigint, pin_sizes, pin_handoff_side_outputs,
        pin_shapes_other_models]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(ORACLE)


# --------------------------------------------------------------------------- planted mistakes (in the oracle, on the CPU)
def _mutant(**overrides):
    m = types.ModuleType("oracle_mutant")
    src = open(ORACLE.__file__).read()
    for old, new in overrides.pop("_edits"):
        assert src.count(old) == 1, old
        src = src.replace(old, new)
    exec(compile(src, "oracle_mutant", "exec"), m.__dict__)
    return m


MUTATIONS = {
    "round_half_up": [("r = np.rint(t).astype(np.float64)", "r = np.floor(t + np.float32(0.5)).astype(np.float64)")],
    "dropped_zero_point_in_code": [("p = r + _per_element(round_zero_point(z), group)", "p = r")],
    "clamp_upper_2^(N-1)": [("q = np.clip(p, 0.0, float(qmax(bits))).astype(np.int32)",
                             "q = np.clip(p, 0.0, float(1 << (bits - 1))).astype(np.int32)")],
    "dequant_sign": [("return (q64 - z64) * s64", "return (q64 + z64) * s64")],
    "ste_frac_sign": [("frac = r - np.asarray(W, np.float64) / s64", "frac = np.asarray(W, np.float64) / s64 - r")],
    "ste_below_above_swapped": [("np.where(below, -z64, Q - z64)", "np.where(below, Q - z64, -z64)")],
    "ste_exclusive_bounds": [("below = p < 0.0", "below = p <= 0.0")],
    "ste_dz_sign": [("clamp_dz = -s64 if dz_mode == 0", "clamp_dz = s64 if dz_mode == 0")],
    "fwd_transposed": [("return np.asarray(X, np.float64) @ np.asarray(W_hat, np.float64).T",
                        "return np.asarray(X, np.float64) @ np.asarray(W_hat, np.float64)")],
    "wgrad_transposed": [("return np.asarray(dY, np.float64).T @ np.asarray(X, np.float64)",
                          "return (np.asarray(X, np.float64).T @ np.asarray(dY, np.float64))")],
    "ds_forgets_zero_point": [("return _group_sum(G * (np.asarray(q, np.float64) - z64), group)",
                               "return _group_sum(G * (np.asarray(q, np.float64)), group)")],
    "pack_msb_first": [('np.packbits(bitplanes.ravel().astype(np.uint8), bitorder="little")',
                        'np.packbits(bitplanes.ravel().astype(np.uint8), bitorder="big")')],
    "real_zero_point_rounded_anyway": [("return np.asarray(z, np.float64) if real_zero_point else round_zero_point(z)",
                                        "return round_zero_point(z)")],
    "minmax_z_sign": [("z = -np.rint(mn / s)", "z = np.rint(mn / s)")],
    "handoff_zero_point_clamp_dropped": [("z8 = np.clip(round_zero_point(z), 0, qmax(bits)).astype(np.uint8)",
                                          "z8 = round_zero_point(z).astype(np.int64).astype(np.uint8)")],
    "handoff_zero_point_truncated": [("z8 = np.clip(round_zero_point(z), 0, qmax(bits)).astype(np.uint8)",
                                      "z8 = np.clip(np.trunc(np.asarray(z, np.float64)), 0, qmax(bits)).astype(np.uint8)")],
    "handoff_step_size_truncated_to_fp16": [("s16 = np.asarray(s, np.float32).astype(np.float16)",
                                             "s16 = (np.ascontiguousarray(s, np.float32).view(np.uint32) & np.uint32(0xFFFFE000))"
                                             ".view(np.float32).astype(np.float16)")],
    "group_sum_wrong_axis": [("return A.reshape(out, in_f // group, group).sum(axis=2, dtype=np.float64)",
                              "return A.reshape(out, group, in_f // group).sum(axis=1, dtype=np.float64)")],
}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name):
    m = _mutant(_edits=MUTATIONS[name])
    caught = []
    for pin in PINS:
        try:
            pin(m)
        except (AssertionError, ValueError):
            caught.append(pin.__name__)
    assert caught, f"no pin notices the planted mistake {name}"
