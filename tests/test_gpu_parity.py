"""Parity of the CUDA library (through its C ABI) with the CPU oracle.

Integer outputs (codes, packed bytes, zero points, fp16 step sizes) must be
bit-exact; floating-point outputs must be within 5e-3 relative Frobenius error
of the oracle (bf16 inputs, fp32 accumulation on the GPU, fp64 in the oracle).
"""
import numpy as np
import pytest
import torch

from helpers import (TOL, Guarded, assert_elementwise, bf16_round, bits_to_torch, contraction_bound, f32, rel_err,
                     torch_to_f64)
from oracle import eqat_oracle as O
from workloads import CONFIGS, Config, Linear, activations_for, get_config, normal_bf16, to_bf16_bits, weight_for

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def eqat():
    from paper_2407_11062_b200.build import build_library
    build_library()
    from paper_2407_11062_b200 import binding
    return binding


@pytest.fixture(autouse=True)
def _device_status_clean(eqat):
    yield
    torch.cuda.synchronize()
    assert eqat.device_status() == (0, 0)


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def small_cfg(name, out, in_f, bits, group, tokens, dist="normal", scale=0.02, outl=0.0):
    return Config(name, (Linear("l", out, in_f, 1),), bits, group, tokens, ("block_ap", "e2e_qp"), dist, scale, outl)


def variants(W32, bits, group):
    """(name, s, z) triples: min/max initialisation, a shrunk step size (forces
    clamping on both sides) and a shifted zero point."""
    s, z = O.minmax_init(W32, bits, group)
    Q = (1 << bits) - 1
    yield "minmax", s, z
    s2 = (s * np.float32(0.7)).astype(np.float32)
    yield "shrunk", s2, z
    yield "shifted", s, np.clip(z + 1, 0, Q).astype(np.float32)


# --------------------------------------------------------------------------- element-wise kernels
@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("group", [32, 64, 128, 256, 512])
def test_minmax_fakequant_ste_pack(eqat, bits, group):
    check_streaming_kernels(eqat, bits, group, 192, 512)      # 98304 elements: twelve tiles of 8192


@pytest.mark.parametrize("out,in_f,bits,group", [
    (1, 128, 2, 64),          # two 128-byte rows: far less than one tile of the copy engine, four live lanes
    (3, 384, 3, 128),         # 1152 elements, 36 live lanes
    (1, 256, 4, 256),         # a single group spread over eight lanes
    (65, 8320, 2, 32),        # 66 tiles and a ragged last one (540800 = 66 * 8192 + 128 elements), groups of 32
    (7, 1152, 2, 1152),       # one group per row, rows that are no power of two (the long-group kernels)
])
def test_streaming_kernels_tiny_and_ragged(eqat, out, in_f, bits, group):
    check_streaming_kernels(eqat, bits, group, out, in_f)


def check_streaming_kernels(eqat, bits, group, out, in_f):
    cfg = small_cfg(f"ew_{bits}_{group}", out, in_f, bits, group, 0, "student_t4", 0.02, 0.01)
    Wb = weight_for(cfg, cfg.linears[0]); W32 = f32(Wb)
    d = eqat.make_desc(bits, group, out, in_f)
    Wd = bits_to_torch(Wb)
    ng = in_f // group

    # min/max initialisation: bit-exact (binary32 arithmetic on both sides)
    s_o, z_o = O.minmax_init(W32, bits, group)
    guard = Guarded()                                    # every output below sits between guard words
    s_g = guard.empty(out, ng); z_g = guard.empty(out, ng)
    eqat.eqat_minmax_init(d, Wd, s_g, z_g)
    assert np.array_equal(s_g.cpu().numpy(), s_o)
    assert np.array_equal(z_g.cpu().numpy(), z_o)

    Gb = normal_bf16((out, in_f), 1e-2, cfg.name, "G"); G32 = f32(Gb); Gd = bits_to_torch(Gb)
    for name, s, z in variants(W32, bits, group):
        sd, zd = dev(s), dev(z)
        q_o, _, p_o = O.quantize_codes(W32, s, z, bits, group)
        if name == "shrunk":
            assert (p_o < 0).any() and (p_o > (1 << bits) - 1).any()       # both clamped branches are exercised
        if name == "shifted":
            assert (p_o > (1 << bits) - 1).any()
        # quantise + pack: bit-exact codes, zero points, fp16 step sizes
        P = guard.empty(out, in_f * bits // 8, dtype=torch.uint8)
        z8 = guard.empty(out, ng, dtype=torch.uint8)
        s16 = guard.empty(out, ng, dtype=torch.float16)
        eqat.eqat_quantize_pack(d, Wd, sd, zd, P, z8, s16)
        P_o, z8_o, s16_o = O.quantize_pack(W32, s, z, bits, group)
        assert np.array_equal(P.cpu().numpy(), P_o), name
        assert np.array_equal(z8.cpu().numpy(), z8_o)
        assert np.array_equal(s16.cpu().numpy().view(np.uint16), s16_o.view(np.uint16))
        # unpack / pack round trip against the oracle's codes
        codes = guard.empty(out, in_f, dtype=torch.uint8)
        eqat.eqat_unpack(d, P, codes)
        assert np.array_equal(codes.cpu().numpy(), q_o.astype(np.uint8))
        P2 = guard.empty(out, in_f * bits // 8, dtype=torch.uint8)
        eqat.eqat_pack(d, dev(q_o.astype(np.uint8)), P2)
        assert np.array_equal(P2.cpu().numpy(), P_o)
        # fake quantiser
        What = guard.empty(out, in_f, dtype=torch.bfloat16)
        eqat.eqat_fakequant_weight(d, Wd, sd, zd, What)
        What_o = O.dequantize(q_o, s, z, group)
        assert rel_err(torch_to_f64(What), What_o) <= TOL
        # the GPU value is the oracle's rounded to bf16, up to one bf16 ulp where the
        # fp32 product sits next to a rounding boundary
        ulp = np.abs(What_o) * 2.0 ** -7 + 1e-30
        assert (np.abs(torch_to_f64(What) - What_o) <= ulp).all()
        # STE backward, both readings of Eq. 4
        for dz_mode in (0, 1):
            dd = eqat.make_desc(bits, group, out, in_f, 0, dz_mode)
            dW = guard.empty(out, in_f, dtype=torch.bfloat16)
            ds = guard.empty(out, ng); dz = guard.empty(out, ng)
            eqat.eqat_ste_bwd(dd, Gd, Wd, sd, zd, dW, ds, dz)
            dW_o, ds_o, dz_o = O.ste_bwd(G32, W32, s, z, bits, group, dz_mode)
            assert np.array_equal(torch_to_f64(dW), dW_o)            # a masked copy: exact
            assert rel_err(torch_to_f64(ds), ds_o) <= TOL, (name, dz_mode)
            if np.linalg.norm(dz_o) > 0:
                assert rel_err(torch_to_f64(dz), dz_o) <= TOL, (name, dz_mode)
            else:
                assert not torch_to_f64(dz).any()
        ds_only = guard.empty(out, ng)
        eqat.eqat_ste_bwd(d, Gd, Wd, sd, zd, dW, ds_only, None)      # dz is optional
        _, ds_o, _ = O.ste_bwd(G32, W32, s, z, bits, group, 0)
        assert rel_err(torch_to_f64(ds_only), ds_o) <= TOL
        guard.check()


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_zero_point_stream(eqat, bits):
    out, in_f, group = 64, 512, 64
    d = eqat.make_desc(bits, group, out, in_f)
    z = np.random.default_rng(bits).integers(0, 1 << bits, out * in_f // group).astype(np.uint8)
    zp = torch.empty(z.size * bits // 8, dtype=torch.uint8, device="cuda")
    eqat.eqat_pack_zeros(d, dev(z), zp)
    assert np.array_equal(zp.cpu().numpy(), O.pack_stream(z, bits))
    back = torch.empty(z.size, dtype=torch.uint8, device="cuda")
    eqat.eqat_unpack_zeros(d, zp, back)
    assert np.array_equal(back.cpu().numpy(), z)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_unpack_into_a_buffer_aligned_to_16_bytes_only(eqat, bits):
    out, in_f, group = 64, 256, 64
    rng = np.random.default_rng(bits)
    q = rng.integers(0, 1 << bits, size=(out, in_f), dtype=np.uint8)
    P = dev(O.pack_rows(q, bits))
    d = eqat.make_desc(bits, group, out, in_f)
    for shift in (0, 16):
        buf = torch.zeros(out * in_f + 32, dtype=torch.uint8, device="cuda")
        codes = buf[shift:shift + out * in_f].view(out, in_f)
        assert codes.data_ptr() % 32 == shift
        eqat.eqat_unpack(d, P, codes)
        assert np.array_equal(codes.cpu().numpy(), q)
        assert not buf[:shift].any() and not buf[shift + out * in_f:].any()


def test_fractional_zero_point_is_rounded(eqat):
    out, in_f, bits, group = 64, 128, 2, 64
    cfg = small_cfg("fracz", out, in_f, bits, group, 0)
    Wb = weight_for(cfg, cfg.linears[0]); W32 = f32(Wb)
    s, z = O.minmax_init(W32, bits, group)
    zf = (z + np.float32(0.3)).astype(np.float32)
    d = eqat.make_desc(bits, group, out, in_f)
    A = torch.empty(out, in_f, dtype=torch.bfloat16, device="cuda"); B = torch.empty_like(A)
    eqat.eqat_fakequant_weight(d, bits_to_torch(Wb), dev(s), dev(z), A)
    eqat.eqat_fakequant_weight(d, bits_to_torch(Wb), dev(s), dev(zf), B)
    assert torch.equal(A, B)


def test_codes_on_exact_and_near_ties(eqat):
    """Quotients that sit exactly on, and a few ulps beside, a rounding boundary:
    w = h * base with h running over integers and half-integers (exact in bf16 for
    a 3-bit base), s = base moved by -3..+3 fp32 ulps.  Codes must equal the
    oracle's (binary32 division, ties to even) on every element."""
    bits, group, in_f = 4, 32, 128
    hs = np.arange(-8.0, 8.5, 0.5, dtype=np.float32)                       # 33 values
    bases = np.array([0.015625, 0.01953125, 0.0234375, 0.02734375, 0.0390625, 0.046875, 0.0546875, 1.25, 0.4375],
                     np.float32)
    rows, s_rows, z_rows = [], [], []
    for base in bases:
        for ulps in range(-3, 4):
            sv = np.float32(base)
            for _ in range(abs(ulps)):
                sv = np.nextafter(sv, np.float32(np.inf if ulps > 0 else -np.inf), dtype=np.float32)
            for zz in (0.0, 7.0):
                rows.append(np.resize(hs * base, in_f).astype(np.float32))
                s_rows.append(np.full(in_f // group, sv, np.float32))
                z_rows.append(np.full(in_f // group, zz, np.float32))
    while len(rows) % 64:
        rows.append(rows[0]); s_rows.append(s_rows[0]); z_rows.append(z_rows[0])
    W32 = np.stack(rows); s = np.stack(s_rows); z = np.stack(z_rows)
    Wb = to_bf16_bits(W32)
    assert np.array_equal(f32(Wb), W32)                                    # the weights are exact in bf16
    out = W32.shape[0]
    d = eqat.make_desc(bits, group, out, in_f)
    P = torch.empty(out, in_f * bits // 8, dtype=torch.uint8, device="cuda")
    z8 = torch.empty(out, in_f // group, dtype=torch.uint8, device="cuda")
    s16 = torch.empty(out, in_f // group, dtype=torch.float16, device="cuda")
    eqat.eqat_quantize_pack(d, bits_to_torch(Wb), dev(s), dev(z), P, z8, s16)
    q_o, _, _ = O.quantize_codes(W32, s, z, bits, group)
    ties = np.abs(np.abs(W32 / np.repeat(s, group, 1)) % 1.0 - 0.5) < 1e-6
    assert ties.sum() > 1000
    codes = torch.empty(out, in_f, dtype=torch.uint8, device="cuda")
    eqat.eqat_unpack(d, P, codes)
    assert np.array_equal(codes.cpu().numpy(), q_o.astype(np.uint8))
    # the fake quantiser and the STE mask take the same decisions
    What = torch.empty(out, in_f, dtype=torch.bfloat16, device="cuda")
    eqat.eqat_fakequant_weight(d, bits_to_torch(Wb), dev(s), dev(z), What)
    assert np.array_equal(torch_to_f64(What), bf16_round(O.dequantize(q_o, s, z, group)).astype(np.float64))
    G = np.ones_like(W32); dW = torch.empty_like(What)
    ds = torch.empty(out, in_f // group, device="cuda")
    eqat.eqat_ste_bwd(d, bits_to_torch(to_bf16_bits(G)), bits_to_torch(Wb), dev(s), dev(z), dW, ds, None)
    dW_o, _, _ = O.ste_bwd(G, W32, s, z, bits, group)
    assert np.array_equal(torch_to_f64(dW), dW_o)


def test_quotients_far_out_of_range_and_zero_points_off_the_grid(eqat):
    """Quotients of magnitude 30 .. 1e30 (and infinite), on and next to half-integers, and zero points far
    outside [0, Q]: the fake-quantised weight and the STE mask must still be the oracle's, element for
    element.  (With a zero point of +-20 or +-40 the in-range window lies around quotients of that size.)"""
    bits, group, in_f = 4, 32, 128
    base = np.float32(0.0234375)
    hs = np.concatenate([np.arange(-45.0, 45.5, 0.5), [31.5, 32.5, 33.5, -32.5, 1e3 + 0.5, -1e4, 3e7, -2e9, 1e30, -1e30]]
                        ).astype(np.float32)
    rows, s_rows, z_rows = [], [], []
    for ulps in range(-2, 3):
        sv = base
        for _ in range(abs(ulps)):
            sv = np.nextafter(sv, np.float32(np.inf if ulps > 0 else -np.inf), dtype=np.float32)
        for zz in (0.0, 15.0, 16.0, 17.0, 20.0, -20.0, 40.0, -40.0):
            for shift in (0, 7, 19):
                rows.append(np.resize(np.roll(hs, shift) * base, in_f).astype(np.float32))
                s_rows.append(np.full(in_f // group, sv, np.float32))
                z_rows.append(np.full(in_f // group, zz, np.float32))
    for big_s, zz in ((1e38, 0.0), (3e38, 7.0)):                           # 1/s is subnormal: no usable reciprocal
        rows.append(np.resize(hs[:181] * np.float32(2e36), in_f).astype(np.float32))   # quotients up to +-0.9 / +-0.3
        s_rows.append(np.full(in_f // group, big_s, np.float32))
        z_rows.append(np.full(in_f // group, zz, np.float32))
    while len(rows) % 64:
        rows.append(rows[0]); s_rows.append(s_rows[0]); z_rows.append(z_rows[0])
    W32 = np.stack(rows); s = np.stack(s_rows); z = np.stack(z_rows)
    Wb = to_bf16_bits(W32); W32 = f32(Wb)                                  # whatever bf16 makes of them
    out = W32.shape[0]
    d = eqat.make_desc(bits, group, out, in_f)
    What = torch.empty(out, in_f, dtype=torch.bfloat16, device="cuda")
    eqat.eqat_fakequant_weight(d, bits_to_torch(Wb), dev(s), dev(z), What)
    # Eq. 2 on the oracle's codes, the product taken in binary32 as the kernel does: with |q - z| up to 40 the
    # product is not exact in binary32, and rounding it to bf16 from binary64 instead could differ in the last bit
    q_o, _, _ = O.quantize_codes(W32, s, z, bits, group)                  # the zero points here are integers
    What_o = bf16_round(((q_o - np.repeat(z, group, 1)).astype(np.float32) * np.repeat(s, group, 1)).astype(np.float32))
    bad = np.argwhere(torch_to_f64(What) != What_o.astype(np.float64))
    assert bad.size == 0, (bad[:5], [(W32[i, j], s[i, j // group], z[i, j // group]) for i, j in bad[:5]])
    # the hand-off takes the same decisions (its exactness test is a different one: two bracketing reciprocals)
    P = torch.empty(out, in_f * bits // 8, dtype=torch.uint8, device="cuda")
    z8 = torch.empty(out, in_f // group, dtype=torch.uint8, device="cuda")
    s16 = torch.empty(out, in_f // group, dtype=torch.float16, device="cuda")
    eqat.eqat_quantize_pack(d, bits_to_torch(Wb), dev(s), dev(z), P, z8, s16)
    codes = torch.empty(out, in_f, dtype=torch.uint8, device="cuda")
    eqat.eqat_unpack(d, P, codes)
    badq = np.argwhere(codes.cpu().numpy() != q_o.astype(np.uint8))
    assert badq.size == 0, (badq[:5], [(W32[i, j], s[i, j // group], z[i, j // group]) for i, j in badq[:5]])
    assert np.array_equal(z8.cpu().numpy(), np.clip(z, 0, (1 << bits) - 1).astype(np.uint8))
    G = np.ones_like(W32); dW = torch.empty_like(What)
    ds = torch.empty(out, in_f // group, device="cuda")
    eqat.eqat_ste_bwd(d, bits_to_torch(to_bf16_bits(G)), bits_to_torch(Wb), dev(s), dev(z), dW, ds, None)
    dW_o, _, _ = O.ste_bwd(G, W32, s, z, bits, group)
    assert np.array_equal(torch_to_f64(dW), dW_o)
    assert dW_o.sum() > 1000 and (dW_o == 0).sum() > 1000                  # both branches well populated


def test_streaming_kernels_repeat_bit_for_bit_on_a_large_weight(eqat):
    """Nine or more tiles per CTA, so every stage of the shared-memory ring is reused several times while the
    consumers run ahead of one another.  A stage that is refilled before all of its readers are done (the
    copy engine's writes are not ordered after ordinary reads without a proxy fence) shows up as a few stale
    rows in some launches, so every kernel is launched a dozen times and must reproduce its first result bit
    for bit; the first result is checked against the oracle on sampled rows."""
    out, in_f, bits, group = 4096, 8192, 2, 64
    ng = in_f // group
    g = torch.Generator(device="cuda"); g.manual_seed(20240711)
    Wd = (torch.randn(out, in_f, device="cuda", generator=g) * 0.02).to(torch.bfloat16)
    Gd = (torch.randn(out, in_f, device="cuda", generator=g) * 0.01).to(torch.bfloat16)
    d = eqat.make_desc(bits, group, out, in_f)

    def run():
        s = torch.empty(out, ng, device="cuda"); z = torch.empty(out, ng, device="cuda")
        eqat.eqat_minmax_init(d, Wd, s, z)
        What = torch.empty(out, in_f, dtype=torch.bfloat16, device="cuda"); dW = torch.empty_like(What)
        ds = torch.empty(out, ng, device="cuda"); dz = torch.empty(out, ng, device="cuda")
        P = torch.empty(out, in_f * bits // 8, dtype=torch.uint8, device="cuda")
        z8 = torch.empty(out, ng, dtype=torch.uint8, device="cuda")
        s16 = torch.empty(out, ng, dtype=torch.float16, device="cuda")
        eqat.eqat_fakequant_weight(d, Wd, s, z, What)
        eqat.eqat_ste_bwd(d, Gd, Wd, s, z, dW, ds, dz)
        eqat.eqat_quantize_pack(d, Wd, s, z, P, z8, s16)
        torch.cuda.synchronize()
        return dict(s=s, z=z, What=What, dW=dW, ds=ds, dz=dz, P=P)

    first = run()
    for _ in range(12):
        again = run()
        for k, v in again.items():
            assert torch.equal(v.view(torch.uint8), first[k].view(torch.uint8)), k
    rows = np.unique(np.concatenate([np.arange(0, out, 97), [out - 1]]))
    W32 = Wd[rows].float().cpu().numpy()
    s_o, z_o = O.minmax_init(W32, bits, group)
    assert np.array_equal(first["s"][rows].cpu().numpy(), s_o) and np.array_equal(first["z"][rows].cpu().numpy(), z_o)
    What_o = O.fake_quant_weight(W32, s_o, z_o, bits, group)              # the oracle's value, to one bf16 ulp
    assert (np.abs(torch_to_f64(first["What"][rows]) - What_o) <= np.abs(What_o) * 2.0 ** -7 + 1e-30).all()
    P_o, _, _ = O.quantize_pack(W32, s_o, z_o, bits, group)
    assert np.array_equal(first["P"][rows].cpu().numpy(), P_o)
    dW_o, ds_o, _ = O.ste_bwd(Gd[rows].float().cpu().numpy(), W32, s_o, z_o, bits, group)
    assert np.array_equal(torch_to_f64(first["dW"][rows]), dW_o)
    assert rel_err(torch_to_f64(first["ds"][rows]), ds_o) <= TOL


# --------------------------------------------------------------------------- Block-AP layer
def workspace_for(eqat, d):
    """Scratch of the Block-AP backward: none (NULL) when the group is reduced inside the GEMM."""
    n = eqat.workspace_bytes(d, eqat.EQAT_OP_FAKEQUANT_BWD)
    assert (n == 0) == (d.group <= 256)
    return torch.empty(n, dtype=torch.uint8, device="cuda") if n else None


def run_block_ap(eqat, cfg, lin, tokens, s, z, dz_mode=0, store_what=True):
    """`store_what=False`: W_hat is not kept; both GEMMs that read it fake-quantise W tile by tile themselves."""
    Wb = weight_for(cfg, lin); Xb, dYb = activations_for(cfg, lin, tokens)
    out, in_f, ng = lin.out_features, lin.in_features, lin.in_features // cfg.group
    d = eqat.make_desc(cfg.bits, cfg.group, out, in_f, tokens, dz_mode)
    Wd, Xd, dYd, sd, zd = bits_to_torch(Wb), bits_to_torch(Xb), bits_to_torch(dYb), dev(s), dev(z)
    guard = Guarded()
    Y = guard.empty(tokens, out, dtype=torch.bfloat16)
    What = guard.empty(out, in_f, dtype=torch.bfloat16) if store_what else None
    eqat.qlinear_fakequant_fwd(d, Xd, Wd, sd, zd, Y, What)
    dX = guard.empty(tokens, in_f, dtype=torch.bfloat16)
    dW = guard.empty(out, in_f, dtype=torch.bfloat16)
    ds = guard.empty(out, ng); dz = guard.empty(out, ng)
    ws = workspace_for(eqat, d)
    eqat.qlinear_fakequant_bwd(d, Xd, dYd, Wd, sd, zd, What, dX, dW, ds, dz, ws)
    guard.check()
    return dict(W=f32(Wb), X=f32(Xb), dY=f32(dYb), Y=Y, What=What, dX=dX, dW=dW, ds=ds, dz=dz)


def check_contractions(r, What_o):
    """Y and dX element by element: each within the rounding a correct kernel can show (see
    helpers.contraction_bound), next to the norm criterion."""
    X, dY = r["X"], r["dY"]
    Y_o, dX_o = O.linear_fwd(X, What_o), O.linear_bwd_dx(dY, What_o)
    assert rel_err(torch_to_f64(r["Y"]), Y_o) <= TOL
    assert rel_err(torch_to_f64(r["dX"]), dX_o) <= TOL
    aW, W2 = np.abs(What_o), What_o ** 2
    assert_elementwise(torch_to_f64(r["Y"]), Y_o,
                       contraction_bound(Y_o, O.linear_fwd(np.abs(X), aW), O.linear_fwd(X ** 2, W2)), "Y")
    assert_elementwise(torch_to_f64(r["dX"]), dX_o,
                       contraction_bound(dX_o, O.linear_bwd_dx(np.abs(dY), aW), O.linear_bwd_dx(dY ** 2, W2)), "dX")


def check_block_ap(r, s, z, bits, group, dz_mode=0):
    What_o = O.fake_quant_weight(r["W"], s, z, bits, group)
    if r["What"] is not None:
        assert rel_err(torch_to_f64(r["What"]), What_o) <= TOL
    check_contractions(r, What_o)
    G = O.weight_grad(r["dY"], r["X"])
    dW_o, ds_o, dz_o = O.ste_bwd(G, r["W"], s, z, bits, group, dz_mode)
    assert rel_err(torch_to_f64(r["dW"]), dW_o) <= TOL
    # dW is the gradient of W_hat, masked, rounded once to bf16 (both operands of its contraction are exact)
    absG = O.weight_grad(np.abs(r["dY"]), np.abs(r["X"]))
    assert_elementwise(torch_to_f64(r["dW"]), dW_o, contraction_bound(dW_o, absG, 0.0, 0), "dW")
    assert rel_err(torch_to_f64(r["ds"]), ds_o) <= TOL
    if np.linalg.norm(dz_o) > 0:
        assert rel_err(torch_to_f64(r["dz"]), dz_o) <= TOL
    else:
        assert not torch_to_f64(r["dz"]).any()


def test_block_ap_config1(eqat):
    cfg = get_config("c1"); lin = cfg.linears[0]
    W32 = f32(weight_for(cfg, lin))
    for name, s, z in variants(W32, cfg.bits, cfg.group):
        for dz_mode in (0, 1):
            r = run_block_ap(eqat, cfg, lin, cfg.tokens, s, z, dz_mode)
            check_block_ap(r, s, z, cfg.bits, cfg.group, dz_mode)


@pytest.mark.parametrize("out,in_f,tokens,bits,group", [
    (192, 384, 300, 4, 128),        # ragged in every dimension: 2 row tiles with a tail, 1.5 column tiles
    (64, 128, 1, 2, 64),            # a single token, a single K block pair
    (320, 640, 129, 3, 128),        # one row past a tile boundary
    (1024, 256, 520, 2, 256),
    (128, 256, 200, 4, 32),         # one 32-column accumulator chunk per group
    (128, 1024, 260, 3, 512),       # groups longer than an output tile: gradient goes through the workspace
    (192, 1024, 64, 2, 1024),       # channel-wise
])
def test_block_ap_ragged(eqat, out, in_f, tokens, bits, group):
    cfg = small_cfg(f"rag_{out}_{in_f}_{tokens}", out, in_f, bits, group, tokens, "student_t4", 0.02, 0.01)
    lin = cfg.linears[0]
    s, z = O.minmax_init(f32(weight_for(cfg, lin)), bits, group)
    s = (s * np.float32(0.8)).astype(np.float32)
    r = run_block_ap(eqat, cfg, lin, tokens, s, z)
    check_block_ap(r, s, z, bits, group)


@pytest.mark.parametrize("out,in_f,tokens,bits,group", [
    (512, 512, 256, 2, 64),         # the first workload's shape: single CTAs
    (512, 512, 700, 4, 128),        # pairs of CTAs, ragged last row-tile
    (192, 384, 300, 3, 32),         # two groups per 64-column unit, ragged in every dimension
    (320, 768, 1030, 2, 256),
    (192, 1408, 600, 4, 1408),      # one group per row, in_features not a power of two
])
def test_block_ap_without_stored_w_hat(eqat, out, in_f, tokens, bits, group):
    """W_hat == NULL: Eq. 1-2 run inside the forward and the dX GEMM on each tile of W.  Same arithmetic as the
    stand-alone fake quantiser, so Y and dX must equal the stored-W_hat form bit for bit, and both match the
    oracle.  The step sizes are shrunk so that both clamped branches (and the exact-division fallback) occur."""
    cfg = small_cfg(f"latent_{out}_{in_f}_{tokens}", out, in_f, bits, group, tokens, "student_t4", 0.02, 0.01)
    lin = cfg.linears[0]
    s, z = O.minmax_init(f32(weight_for(cfg, lin)), bits, group)
    s = (s * np.float32(0.8)).astype(np.float32)
    a = run_block_ap(eqat, cfg, lin, tokens, s, z, store_what=True)
    b = run_block_ap(eqat, cfg, lin, tokens, s, z, store_what=False)
    check_block_ap(b, s, z, bits, group)
    for k in ("Y", "dX", "dW", "ds", "dz"):
        assert torch.equal(a[k], b[k]), k


def test_outputs_aligned_to_16_bytes_only(eqat):
    """Outputs need 16-byte alignment only: the same bits at a 16-byte offset from a 512-byte boundary."""
    cfg = get_config("c1"); lin = cfg.linears[0]
    out, in_f, T = lin.out_features, lin.in_features, cfg.tokens
    s, z = O.minmax_init(f32(weight_for(cfg, lin)), cfg.bits, cfg.group)
    Wd = bits_to_torch(weight_for(cfg, lin)); Xb, dYb = activations_for(cfg, lin, T)
    Xd, dYd, sd, zd = bits_to_torch(Xb), bits_to_torch(dYb), dev(s), dev(z)
    d = eqat.make_desc(cfg.bits, cfg.group, out, in_f, T)
    What = torch.empty(out, in_f, dtype=torch.bfloat16, device="cuda")
    ws = workspace_for(eqat, d)
    res = []
    for shift in (0, 8):                                         # elements: 0 or 16 bytes past a 512-byte boundary
        Y = torch.zeros(T * out + 16, dtype=torch.bfloat16, device="cuda")[shift:shift + T * out].view(T, out)
        dX = torch.zeros(T * in_f + 16, dtype=torch.bfloat16, device="cuda")[shift:shift + T * in_f].view(T, in_f)
        dW = torch.zeros(out * in_f + 16, dtype=torch.bfloat16, device="cuda")[shift:shift + out * in_f].view(out, in_f)
        assert Y.data_ptr() % 32 == 2 * shift
        ds = torch.empty(out, in_f // cfg.group, device="cuda"); dz = torch.empty_like(ds)
        eqat.qlinear_fakequant_fwd(d, Xd, Wd, sd, zd, Y, What)
        eqat.qlinear_fakequant_bwd(d, Xd, dYd, Wd, sd, zd, What, dX, dW, ds, dz, ws)
        torch.cuda.synchronize()
        res.append((Y.clone(), dX.clone(), dW.clone()))
    for a, b in zip(*res):
        assert torch.equal(a, b)


def test_block_ap_is_deterministic(eqat):
    cfg = get_config("c1"); lin = cfg.linears[0]
    s, z = O.minmax_init(f32(weight_for(cfg, lin)), cfg.bits, cfg.group)
    a = run_block_ap(eqat, cfg, lin, cfg.tokens, s, z)
    b = run_block_ap(eqat, cfg, lin, cfg.tokens, s, z)
    for k in ("Y", "What", "dX", "dW", "ds", "dz"):
        assert torch.equal(a[k], b[k]), k


# --------------------------------------------------------------------------- E2E-QP layer
def run_e2e(eqat, cfg, lin, tokens, with_dz=True, fp16_steps=False, real_z=False):
    """Hand-off (quantise + pack on the oracle's side) then the three packed-weight calls.  `real_z`: the zero
    points are handed over as fp16 values moved off the integers (the variant that trains z), codes unchanged."""
    Wb = weight_for(cfg, lin); W32 = f32(Wb)
    Xb, dYb = activations_for(cfg, lin, tokens)
    out, in_f, ng = lin.out_features, lin.in_features, lin.in_features // cfg.group
    s, z = O.minmax_init(W32, cfg.bits, cfg.group)
    if fp16_steps:
        s = s.astype(np.float16).astype(np.float32)
    P_o, z8_o, s16_o = O.quantize_pack(W32, s, z, cfg.bits, cfg.group)
    zfmt = eqat.EQAT_ZP_FP16 if real_z else eqat.EQAT_ZP_U8
    d = eqat.make_desc(cfg.bits, cfg.group, out, in_f, tokens, 0, zfmt)
    if real_z:
        drift = np.random.default_rng(ng + out).uniform(-0.45, 0.45, z8_o.shape)
        z_o = (z8_o + drift).astype(np.float16)                          # what a few optimiser steps leave behind
        zd = torch.from_numpy(z_o.view(np.int16)).view(torch.float16).cuda()
        z_o = z_o.astype(np.float32)
    else:
        z_o, zd = z8_o, dev(z8_o)
    Pd = dev(P_o)
    s16d = torch.from_numpy(s16_o.view(np.int16)).view(torch.float16).cuda()
    Xd, dYd = bits_to_torch(Xb), bits_to_torch(dYb)
    guard = Guarded()
    Y = guard.empty(tokens, out, dtype=torch.bfloat16)
    dX = guard.empty(tokens, in_f, dtype=torch.bfloat16)
    ds = guard.empty(out, ng)
    dz = guard.empty(out, ng) if with_dz else None
    n_ws = eqat.workspace_bytes(d, eqat.EQAT_OP_PACKED_BWD_DS)
    assert (n_ws > 0) == (cfg.group > 256)                               # only one group per row needs scratch
    ws = guard.empty(n_ws, dtype=torch.uint8) if n_ws else None
    eqat.qlinear_packed_fwd(d, Xd, Pd, s16d, zd, Y)
    eqat.qlinear_packed_bwd_dx(d, dYd, Pd, s16d, zd, dX)
    eqat.qlinear_packed_bwd_ds(d, Xd, dYd, Pd, zd, s16d, ds, dz, ws)
    guard.check()
    q = O.unpack_rows(P_o, cfg.bits, in_f)
    return dict(X=f32(Xb), dY=f32(dYb), q=q, z8=z_o, s16=s16_o.astype(np.float32), Y=Y, dX=dX, ds=ds, dz=dz,
                W=W32, s=s, z=z, real_z=real_z)


def check_e2e(r, group):
    rz = r["real_z"]
    What_o = O.dequantize(r["q"], r["s16"], r["z8"], group, real_zero_point=rz)
    check_contractions(r, What_o)
    assert rel_err(torch_to_f64(r["ds"]), O.e2e_ds(r["dY"], r["X"], r["q"], r["z8"], group, real_zero_point=rz)) <= TOL
    if r["dz"] is not None:
        assert rel_err(torch_to_f64(r["dz"]), O.e2e_dz(r["dY"], r["X"], r["s16"], group)) <= TOL


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("group", [32, 64, 128, 256, 512])
@pytest.mark.parametrize("real_z", [False, True], ids=["z_u8", "z_fp16"])
def test_e2e_small(eqat, bits, group, real_z):
    """Every group size of the paper's ablation (32 .. 256) and one group per row (512 = in_features, the
    channel-wise setting of its Q-PEFT comparison), with frozen integer zero points and with trained fp16 ones.
    600 tokens: a pair of CTAs per tile with a ragged last row-tile; 256: single CTAs."""
    for tokens in (600, 256):
        cfg = small_cfg(f"e2e_{bits}_{group}", 512, 512, bits, group, tokens, "student_t4", 0.02, 0.01)
        check_e2e(run_e2e(eqat, cfg, cfg.linears[0], tokens, real_z=real_z), group)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("tokens", [1, 2, 3, 4, 5, 7, 8, 9])
def test_e2e_few_tokens(eqat, bits, tokens):
    """Decode-sized batches: up to eight tokens take a matrix-vector forward kernel, more the tiled one (rows this
    short are not worth several launches).
    640 = 10 units of 64 columns, fewer than the sixteen warps of a CTA (some get none); 1408 = 22 (one or two each)."""
    group = 64 if bits == 2 else 128
    cfg = small_cfg(f"gemv_{bits}_{tokens}", 448, 640 if group == 64 else 1408, bits, group, tokens, "student_t4", 0.02, 0.01)
    check_e2e(run_e2e(eqat, cfg, cfg.linears[0], tokens), group)


@pytest.mark.parametrize("bits,group,in_f,tokens", [
    (2, 64, 1024, 1),       # four groups of 64 per 256 columns, vector loads of the parameters
    (2, 64, 4096, 13),      # sliced: seven and six tokens
    (3, 128, 2048, 5),      # two groups of 128 per 256 columns
    (4, 128, 1408, 8),      # an odd number of groups per row: parameters fetched chunk by chunk
    (2, 256, 1024, 3),      # one group per 256 columns
    (4, 1152, 1152, 2),     # one group per row
])
def test_e2e_few_tokens_with_trained_zero_points(eqat, bits, group, in_f, tokens):
    """The matrix-vector forward with fp16 zero points off the integers (the variant that trains z)."""
    cfg = small_cfg(f"gemv_rz_{bits}_{group}_{tokens}", 320, in_f, bits, group, tokens, "student_t4", 0.02, 0.01)
    check_e2e(run_e2e(eqat, cfg, cfg.linears[0], tokens, real_z=True), group)


def test_few_token_forward_agrees_with_tiled_forward(eqat):
    """The same rows through both forward kernels (4 tokens alone, and as the first rows of a 9-token batch)."""
    cfg = small_cfg("gemv_vs_gemm", 512, 1024, 2, 64, 9)
    r5 = run_e2e(eqat, cfg, cfg.linears[0], 9)
    cfg4 = small_cfg("gemv_vs_gemm", 512, 1024, 2, 64, 4)
    Wb = weight_for(cfg4, cfg4.linears[0])
    assert np.array_equal(Wb, weight_for(cfg, cfg.linears[0]))
    P_o, z8_o, s16_o = O.quantize_pack(r5["W"], r5["s"], r5["z"], 2, 64)
    X4 = torch.from_numpy(bf16_round(r5["X"][:4]).astype(np.float32)).to(torch.bfloat16).cuda()
    d = eqat.make_desc(2, 64, 512, 1024, 4)
    Y4 = torch.empty(4, 512, dtype=torch.bfloat16, device="cuda")
    s16d = torch.from_numpy(s16_o.view(np.int16)).view(torch.float16).cuda()
    eqat.qlinear_packed_fwd(d, X4, dev(P_o), s16d, dev(z8_o), Y4)
    torch.cuda.synchronize()
    assert rel_err(torch_to_f64(Y4), torch_to_f64(r5["Y"][:4])) <= TOL


@pytest.mark.parametrize("bits,group", [(2, 64), (3, 128), (3, 64), (4, 128), (4, 64)])
def test_few_token_forward_is_deterministic(eqat, bits, group):
    """More row-blocks than SMs, several stages per row-block: the partial sums of the sixteen warps are added in
    a fixed order by one warp, so repeated launches must agree bit for bit (also while other work runs beside them)."""
    out, in_f, T = 2432, 5120, 3
    g = torch.Generator(device="cuda"); g.manual_seed(11)
    P = torch.randint(0, 256, (out, in_f * bits // 8), dtype=torch.uint8, device="cuda", generator=g)
    z8 = torch.randint(0, 1 << bits, (out, in_f // group), dtype=torch.uint8, device="cuda", generator=g)
    s16 = (torch.rand(out, in_f // group, device="cuda", generator=g) * 0.01 + 0.001).half()
    X = torch.randn(T, in_f, device="cuda", generator=g).to(torch.bfloat16)
    d = eqat.make_desc(bits, group, out, in_f, T)
    ref = torch.empty(T, out, dtype=torch.bfloat16, device="cuda")
    eqat.qlinear_packed_fwd(d, X, P, s16, z8, ref)
    side = torch.cuda.Stream()
    noise = torch.empty(1 << 26, device="cuda")
    for _ in range(5):
        with torch.cuda.stream(side):
            noise.normal_()                                # unrelated traffic on another stream
        Y = torch.full_like(ref, float("nan"))
        eqat.qlinear_packed_fwd(d, X, P, s16, z8, Y)
        torch.cuda.synchronize()
        assert torch.equal(Y.view(torch.int16), ref.view(torch.int16))
    # and it is the right answer
    q = O.unpack_rows(P.cpu().numpy(), bits, in_f)
    What_o = O.dequantize(q, s16.cpu().numpy().astype(np.float32), z8.cpu().numpy(), group)
    assert rel_err(torch_to_f64(ref), O.linear_fwd(torch_to_f64(X), What_o)) <= TOL


def few_token_problem(out, in_f, tokens, seed, bits=2, group=64):
    """Random packed bytes (every code value equally likely), zero points near the middle of the code range."""
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    Q = (1 << bits) - 1
    P = torch.randint(0, 256, (out, in_f * bits // 8), dtype=torch.uint8, device="cuda", generator=g)
    z8 = torch.randint(Q // 2, Q // 2 + 2, (out, in_f // group), dtype=torch.uint8, device="cuda", generator=g)
    s16 = ((torch.rand(out, in_f // group, device="cuda", generator=g) * 0.004 + 0.012) * 3 / Q).half()
    X = torch.randn(tokens, in_f, device="cuda", generator=g).to(torch.bfloat16)
    return P, z8, s16, X


@pytest.mark.parametrize("bits,group", [(2, 64), (3, 128), (4, 128)])
def test_few_token_forward_does_not_depend_on_the_slicing(eqat, bits, group):
    """Thirteen tokens go out as two launches (seven and six tokens); every token's row must be bit for bit what the
    token gives alone, and what it gives in a batch of eight (one launch)."""
    out, in_f, T = 1280, 4096, 13
    P, z8, s16, X = few_token_problem(out, in_f, T, 21, bits, group)
    guard = Guarded()
    Y = guard.empty(T, out, dtype=torch.bfloat16)
    eqat.qlinear_packed_fwd(eqat.make_desc(bits, group, out, in_f, T), X, P, s16, z8, Y)
    Y8 = guard.empty(8, out, dtype=torch.bfloat16)
    eqat.qlinear_packed_fwd(eqat.make_desc(bits, group, out, in_f, 8), X[:8].contiguous(), P, s16, z8, Y8)
    guard.check()
    assert torch.equal(Y8.view(torch.int16), Y[:8].view(torch.int16))
    d1 = eqat.make_desc(bits, group, out, in_f, 1)
    for t in range(T):
        y = torch.empty(1, out, dtype=torch.bfloat16, device="cuda")
        eqat.qlinear_packed_fwd(d1, X[t:t + 1].contiguous(), P, s16, z8, y)
        torch.cuda.synchronize()
        assert torch.equal(y.view(torch.int16), Y[t:t + 1].view(torch.int16)), t
    q = O.unpack_rows(P.cpu().numpy(), bits, in_f)
    What_o = O.dequantize(q, s16.cpu().numpy().astype(np.float32), z8.cpu().numpy(), group)
    assert rel_err(torch_to_f64(Y), O.linear_fwd(torch_to_f64(X), What_o)) <= TOL


@pytest.mark.parametrize("bits,group,tokens", [(2, 64, 1), (2, 64, 8), (2, 64, 12), (3, 128, 5), (4, 128, 3), (4, 128, 12)])
def test_few_token_forwards_back_to_back_keep_their_order(eqat, bits, group, tokens):
    """Twelve layers in a row, each reading what the one before wrote, issued without a pause (the launches may
    overlap their start-up with the tail of the launch before) and again with a synchronise after every call."""
    n = 4096
    Ps = [few_token_problem(n, n, tokens, 30 + i, bits, group)[0] for i in range(12)]
    _, z8, s16, X0 = few_token_problem(n, n, tokens, 29, bits, group)
    d = eqat.make_desc(bits, group, n, n, tokens)

    def chain(pause):
        bufs = [X0.clone(), torch.zeros_like(X0)]
        for i, P in enumerate(Ps):
            eqat.qlinear_packed_fwd(d, bufs[i & 1], P, s16, z8, bufs[(i + 1) & 1])
            if pause:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        return bufs[len(Ps) & 1].clone()

    ref = chain(True)
    assert torch.isfinite(ref.float()).all() and float(ref.float().abs().max()) > 1e-3
    for _ in range(10):
        assert torch.equal(chain(False).view(torch.int16), ref.view(torch.int16))
    assert eqat.device_status() == (0, 0)


@pytest.mark.parametrize("out,in_f,tokens,bits,group", [
    (192, 384, 300, 2, 64),
    (64, 128, 1, 4, 128),
    (320, 640, 129, 3, 128),
    (1024, 256, 520, 2, 64),
    (64, 11008, 4, 2, 64),          # few-token kernel with more than 48 KB of staged activations
    (64, 28672, 2, 4, 128),         # the longest rows of the 70B block, 4-bit codes: two tokens fit one launch
    (64, 28672, 3, 3, 128),         # 3-bit codes, the longest rows: slices of two tokens and one
    (448, 1408, 700, 3, 32),        # groups of 32, nothing a multiple of a tile
    (320, 1408, 1100, 2, 1408),     # one group per row with in_features not a power of two: 5.5 column tiles
    (192, 640, 3, 4, 640),          # one group per row through the few-token kernel
    (192, 640, 3, 2, 32),           # groups of 32 with few tokens: the tiled kernel
    (128, 1152, 3, 2, 1152),        # 2-bit codes, one group per row, few tokens: the tensor-core matrix-vector kernel
    (192, 768, 2, 2, 128),          # the same kernel with groups of 128 (two 64-column chunks per group) ...
    (80 * 16, 4608, 1, 2, 256),     # ... and of 256; 80 row-blocks of 16 over several stages of the ring, 9 boxes per row
    (64, 128, 1, 2, 64),            # rows of 32 bytes: a quarter of the copy engine's 128-byte box
    (64, 256, 8, 2, 128),           # eight tokens, the most the matrix-vector kernel takes
    (2432, 512, 4, 2, 64),          # more row-blocks than SMs: every CTA takes a second task, parameters loaded as vectors
    (64, 11008, 8, 2, 64),          # eight tokens whose staged activations do not fit: two launches of four
    (128, 4096, 13, 2, 64),         # more than eight tokens: slices of seven and six
    (128, 8192, 31, 2, 128),        # five slices (7, 7, 7, 7, 3)
    (64, 28672, 4, 2, 64),          # the longest rows of the 70B block: two tokens per launch
    (64, 11008, 8, 4, 128),         # 4-bit codes: 43 boxes of 256 columns per row, two launches of four tokens
    (128, 4096, 13, 4, 64),         # 4-bit codes, groups of 64 (one group per chunk), slices of seven and six
    (80 * 16, 2304, 5, 4, 256),     # 4-bit codes, groups of 256, nine boxes per row, 80 row-blocks
    (64, 128, 2, 4, 64),            # rows of 64 bytes: half a box, two chunks, two groups
    (128, 4096, 13, 3, 128),        # 3-bit codes: boxes of 96 bytes (256 columns), slices of seven and six
    (80 * 16, 2304, 5, 3, 256),     # 3-bit codes, groups of 256, nine boxes per row, 80 row-blocks
    (64, 11008, 8, 3, 64),          # 3-bit codes, groups of 64, 43 boxes per row, two launches of four tokens
    (64, 128, 1, 3, 128),           # 3-bit rows of 48 bytes: half a box, one group
    (128, 11008, 40, 2, 64),        # forty tokens over long rows: eight launches of five
    (128, 11008, 64, 4, 128),       # the most tokens that go out in slices: thirteen launches (twelve of five, one of four)
])
def test_e2e_ragged(eqat, out, in_f, tokens, bits, group):
    cfg = small_cfg(f"e2er_{out}_{in_f}_{tokens}", out, in_f, bits, group, tokens)
    check_e2e(run_e2e(eqat, cfg, cfg.linears[0], tokens, with_dz=(bits != 4), real_z=(group in (32, 640))), group)


def test_e2e_is_deterministic_and_matches_block_ap_forward(eqat):
    """Packed forward == fake-quant forward when s is representable in fp16."""
    cfg = small_cfg("cross", 512, 512, 2, 64, 256)
    lin = cfg.linears[0]
    a = run_e2e(eqat, cfg, lin, 256, fp16_steps=True)
    b = run_e2e(eqat, cfg, lin, 256, fp16_steps=True)
    for k in ("Y", "dX", "ds", "dz"):
        assert torch.equal(a[k], b[k]), k
    assert np.array_equal(a["s"], a["s16"])       # the step sizes survive the fp16 hand-off unchanged
    r = run_block_ap(eqat, cfg, lin, 256, a["s"], a["z"])
    assert rel_err(torch_to_f64(r["Y"]), torch_to_f64(a["Y"])) <= 2e-3
    assert rel_err(torch_to_f64(r["dX"]), torch_to_f64(a["dX"])) <= 2e-3


# --------------------------------------------------------------------------- hand-off side outputs, alignment, waits
@pytest.mark.parametrize("kind,bits", [("z2", 2), ("z4", 4)])
def test_handoff_side_outputs_against_hand_values(eqat, kind, bits):
    """Step sizes that fp16 cannot hold exactly and zero points that are fractional or outside [0, Q]: the fp16
    bit patterns and the stored bytes are the hand-derived ones of tests/golden/handoff_side_outputs.txt (the
    same fixture pins the oracle), through both quantise + pack kernels (groups of 32 and channel-wise)."""
    import os
    from conftest import GOLDEN
    rows = [[x.strip() for x in l.split("|")] for l in open(os.path.join(GOLDEN, "handoff_side_outputs.txt"))
            if l.strip() and not l.startswith("#")]
    s_rows = [(float(v), int(h, 16)) for k, v, h in rows if k == "s"]
    z_rows = [(float(v), int(b)) for k, v, b in rows if k == kind]
    for group, in_f in ((32, 128), (512, 512)):
        ng, out = in_f // group, 8
        s = np.array([[s_rows[(o + j) % 4][0] for j in range(ng)] for o in range(out)], np.float32)
        s_bits = np.array([[s_rows[(o + j) % 4][1] for j in range(ng)] for o in range(out)], np.uint16)
        z = np.array([[z_rows[(o + j) % len(z_rows)][0] for j in range(ng)] for o in range(out)], np.float32)
        z_bytes = np.array([[z_rows[(o + j) % len(z_rows)][1] for j in range(ng)] for o in range(out)], np.uint8)
        Wb = normal_bf16((out, in_f), 0.05, "handoff", kind, group)
        d = eqat.make_desc(bits, group, out, in_f)
        guard = Guarded()
        P = guard.empty(out, in_f * bits // 8, dtype=torch.uint8)
        z8 = guard.empty(out, ng, dtype=torch.uint8)
        s16 = guard.empty(out, ng, dtype=torch.float16)
        eqat.eqat_quantize_pack(d, bits_to_torch(Wb), dev(s), dev(z), P, z8, s16)
        guard.check()
        assert np.array_equal(z8.cpu().numpy(), z_bytes)
        assert np.array_equal(s16.cpu().numpy().view(np.uint16), s_bits)
        P_o, z8_o, s16_o = O.quantize_pack(f32(Wb), s, z, bits, group)
        assert np.array_equal(P.cpu().numpy(), P_o)
        assert np.array_equal(z8_o, z_bytes) and np.array_equal(s16_o.view(np.uint16), s_bits)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("tokens", [1, 4, 300])
def test_packed_weight_aligned_to_16_bytes_only(eqat, bits, tokens):
    """The packed matrix (and its step sizes and zero points) 16 bytes past a 256-byte boundary: 16-byte alignment is
    all the interface asks for, so the kernels must not fetch whole 32-byte sectors from it.  Same bits as the
    aligned run, through the matrix-vector kernel (1 and 4 tokens) and the tiled one."""
    group = 64 if bits == 2 else 128
    cfg = small_cfg(f"wq16_{bits}", 320, 512, bits, group, tokens, "student_t4", 0.02, 0.01)
    lin = cfg.linears[0]
    out, in_f, ng = 320, 512, 512 // group
    W32 = f32(weight_for(cfg, lin))
    s, z = O.minmax_init(W32, bits, group)
    P_o, z8_o, s16_o = O.quantize_pack(W32, s, z, bits, group)
    Xb, dYb = activations_for(cfg, lin, tokens)
    Xd, dYd = bits_to_torch(Xb), bits_to_torch(dYb)
    d = eqat.make_desc(bits, group, out, in_f, tokens)
    res = []
    for shift in (0, 16):
        def place(a):
            raw = torch.zeros(a.nbytes + 32, dtype=torch.uint8, device="cuda")
            v = raw[shift:shift + a.nbytes]
            v.copy_(torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).ravel()))
            assert v.data_ptr() % 32 == shift
            return v
        Pd, z8d, s16d = place(P_o), place(z8_o), place(s16_o)
        guard = Guarded()
        Y = guard.empty(tokens, out, dtype=torch.bfloat16)
        dX = guard.empty(tokens, in_f, dtype=torch.bfloat16)
        ds = guard.empty(out, ng)
        eqat.qlinear_packed_fwd(d, Xd, Pd, s16d, z8d, Y)
        eqat.qlinear_packed_bwd_dx(d, dYd, Pd, s16d, z8d, dX)
        eqat.qlinear_packed_bwd_ds(d, Xd, dYd, Pd, z8d, s16d, ds)
        guard.check()
        res.append((Y.clone(), dX.clone(), ds.clone()))
    for a, b in zip(*res):
        assert torch.equal(a, b)
    q = O.unpack_rows(P_o, bits, in_f)
    What_o = O.dequantize(q, s16_o.astype(np.float32), z8_o, group)
    assert rel_err(torch_to_f64(res[1][0]), O.linear_fwd(f32(Xb), What_o)) <= TOL


def test_block_level_calls_equal_the_layer_calls(eqat):
    """eqat_block_ap_step and eqat_e2e_qp_step over three linears of different shapes (one with one group per row,
    which needs both kinds of scratch): bit for bit what the layer entry points give, called one by one."""
    specs = [(256, 512, 300, 64), (192, 384, 300, 128), (128, 640, 300, 640)]
    bits = 2
    ap_rows, e2e_rows, expect = [], [], []
    for k, (out, in_f, T, group) in enumerate(specs):
        cfg = small_cfg(f"blk_{k}", out, in_f, bits, group, T, "student_t4", 0.02, 0.01)
        lin = cfg.linears[0]
        ng = in_f // group
        W32 = f32(weight_for(cfg, lin)); Xb, dYb = activations_for(cfg, lin, T)
        s, z = O.minmax_init(W32, bits, group)
        P_o, z8_o, s16_o = O.quantize_pack(W32, s, z, bits, group)
        Wd, Xd, dYd, sd, zd = bits_to_torch(weight_for(cfg, lin)), bits_to_torch(Xb), bits_to_torch(dYb), dev(s), dev(z)
        Pd, z8d = dev(P_o), dev(z8_o)
        s16d = torch.from_numpy(s16_o.view(np.int16)).view(torch.float16).cuda()
        d = eqat.make_desc(bits, group, out, in_f, T)
        bf = torch.bfloat16

        def outs_ap():
            n = eqat.workspace_bytes(d, eqat.EQAT_OP_FAKEQUANT_BWD)
            return dict(Y=torch.empty(T, out, dtype=bf, device="cuda"), W_hat=torch.empty(out, in_f, dtype=bf, device="cuda"),
                        dX=torch.empty(T, in_f, dtype=bf, device="cuda"), dW=torch.empty(out, in_f, dtype=bf, device="cuda"),
                        ds=torch.empty(out, ng, device="cuda"), dz=torch.empty(out, ng, device="cuda"),
                        workspace=torch.empty(n, dtype=torch.uint8, device="cuda") if n else None)

        def outs_e2e():
            n = eqat.workspace_bytes(d, eqat.EQAT_OP_PACKED_BWD_DS)
            return dict(Y=torch.empty(T, out, dtype=bf, device="cuda"), dX=torch.empty(T, in_f, dtype=bf, device="cuda"),
                        ds=torch.empty(out, ng, device="cuda"), dz=torch.empty(out, ng, device="cuda"),
                        workspace=torch.empty(n, dtype=torch.uint8, device="cuda") if n else None)

        a, b = outs_ap(), outs_ap()
        eqat.qlinear_fakequant_fwd(d, Xd, Wd, sd, zd, a["Y"], a["W_hat"])
        eqat.qlinear_fakequant_bwd(d, Xd, dYd, Wd, sd, zd, a["W_hat"], a["dX"], a["dW"], a["ds"], a["dz"], a["workspace"])
        ap_rows.append(dict(desc=d, X=Xd, dY=dYd, W=Wd, s=sd, z=zd, **b))
        c, e = outs_e2e(), outs_e2e()
        eqat.qlinear_packed_fwd(d, Xd, Pd, s16d, z8d, c["Y"])
        eqat.qlinear_packed_bwd_dx(d, dYd, Pd, s16d, z8d, c["dX"])
        eqat.qlinear_packed_bwd_ds(d, Xd, dYd, Pd, z8d, s16d, c["ds"], c["dz"], c["workspace"])
        e2e_rows.append(dict(desc=d, X=Xd, dY=dYd, Wq_packed=Pd, s16=s16d, z=z8d, **e))
        expect.append((a, c))
    eqat.eqat_block_ap_step(ap_rows)
    eqat.eqat_e2e_qp_step(e2e_rows)
    torch.cuda.synchronize()
    for (a, c), got_ap, got_e2e in zip(expect, ap_rows, e2e_rows):
        for k in ("Y", "W_hat", "dX", "dW", "ds", "dz"):
            assert torch.equal(got_ap[k], a[k]), k
        for k in ("Y", "dX", "ds", "dz"):
            assert torch.equal(got_e2e[k], c[k]), k
    # a fault in the last linear: reported with its index, and nothing has run (the first linear's outputs keep
    # the pattern they are given here)
    ap_rows[0]["Y"].fill_(7.0)
    broken = [dict(r) for r in ap_rows]
    broken[2]["dW"] = None
    with pytest.raises(eqat.EqatError, match="linear 2") as err:
        eqat.eqat_block_ap_step(broken)
    assert err.value.status == eqat.EQAT_ERR_NULL
    torch.cuda.synchronize()
    assert bool((ap_rows[0]["Y"] == 7.0).all())


@pytest.mark.parametrize("which,name", [(0, "GEMM kernels"), (1, "streaming kernels"), (2, "matrix-vector kernel")])
def test_a_bounded_wait_runs_out_cleanly(eqat, which, name):
    """One warp waits 1 ms for a barrier that nothing signals, through the kernels' own wait routine: the kernel
    must end normally, the status word must say TIMEOUT with the self-test's site code exactly once, and the
    library must work afterwards (the context is intact)."""
    torch.cuda.synchronize()
    assert eqat.device_status() == (0, 0)
    eqat.eqat_selftest_wait_expiry(which)
    torch.cuda.synchronize()                                   # the kernel returned: no hang, no fault
    assert eqat.device_status() == (eqat.EQAT_ERR_TIMEOUT, 9)
    assert eqat.device_status() == (0, 0)                      # reading clears it
    cfg = get_config("c1"); lin = cfg.linears[0]
    s, z = O.minmax_init(f32(weight_for(cfg, lin)), cfg.bits, cfg.group)
    check_block_ap(run_block_ap(eqat, cfg, lin, cfg.tokens, s, z), s, z, cfg.bits, cfg.group)
