"""Parity at the full sizes of the five workloads, in the launch configuration
the benchmark times (one call per linear, whole matrices).

The oracle cannot form 10^13-flop products, so each floating-point output is
compared on a seeded sample it can compute directly:
  * Y on 192 token rows x 256 output rows, dX on 192 token rows x 4 column groups,
  * dW / ds / dz (and the packed ds) on 96 output rows x all columns,
  * codes, packed bytes, zero points and step sizes bit-exactly on those rows,
each sampled block by its norm and element by element (helpers.contraction_bound); a second, dense block
always covers the last row-tile and the last column-tile of Y and dX (last 256 tokens x last 256 outputs /
inputs), where a ragged edge would show; and whole-tensor identities that hold at any size tie the rest together:
  <dY, Y> = <dX, X>  (adjoint),  sum s*ds = <dY, Y>  (Y is linear in s).
The E2E-QP cases also push the first 1, 4, 8 and 20 tokens through the forward alone (decoding).
"""
import numpy as np
import pytest
import torch

from helpers import TOL, assert_elementwise, bits_to_torch, contraction_bound, f32, rel_err, torch_to_f64
from oracle import eqat_oracle as O
from workloads import CONFIGS, activations_for, get_config, tensor_seed, weight_for

pytestmark = pytest.mark.gpu

N_TOK, N_OUT_Y, N_OUT_G, N_COL_GROUPS = 192, 256, 96, 4


@pytest.fixture(scope="module")
def eqat():
    from paper_2407_11062_b200.build import build_library
    build_library()
    from paper_2407_11062_b200 import binding
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def sample(n, k, *key):
    rng = np.random.default_rng(tensor_seed(*key) % (2 ** 32))
    idx = np.sort(rng.choice(n, size=min(k, n), replace=False))
    idx[0], idx[-1] = 0, n - 1                      # always include the first and the last row
    return np.unique(idx)


def dot64(a: torch.Tensor, b: torch.Tensor) -> float:
    """<a, b> over whole device tensors, accumulated in float64 in row blocks."""
    tot = 0.0
    step = max(1, (1 << 24) // a.shape[1])
    for i in range(0, a.shape[0], step):
        tot += float((a[i:i + step].double() * b[i:i + step].double()).sum())
    return tot


def inner_product_tol(dY, Y, dX, X) -> float:
    """Allowed gap between <dY, Y> and <dX, X>.  Both are sums of n zero-mean
    products, so their size is about |u||v|/sqrt(n); element errors of relative
    size e perturb them by about e|u||v|/sqrt(n).  The bound is TOL times that
    scale for each side."""
    def scale(u, v):
        return np.sqrt(dot64(u, u) * dot64(v, v) / u.numel())
    return TOL * (scale(dY, Y) + scale(dX, X))


def check_block(got, A, B_rows, what):
    """got ~ A @ B_rows.T for the oracle's operands (fp64): norm criterion and element-wise bound."""
    ref = O.linear_fwd(A, B_rows)
    assert rel_err(torch_to_f64(got), ref) <= TOL, what
    bound = contraction_bound(ref, O.linear_fwd(np.abs(A), np.abs(B_rows)), O.linear_fwd(A ** 2, B_rows ** 2))
    assert_elementwise(torch_to_f64(got), ref, bound, what)


CORNER = 256


CASES = [(c.name, l.name, mode) for c in CONFIGS[1:] for l in c.linears for mode in c.modes]


@pytest.mark.parametrize("cfg_name,lin_name,mode", CASES)
def test_full_size(eqat, cfg_name, lin_name, mode):
    cfg = get_config(cfg_name)
    lin = next(l for l in cfg.linears if l.name == lin_name)
    out, in_f, T, bits, g = lin.out_features, lin.in_features, cfg.tokens, cfg.bits, cfg.group
    ng = in_f // g
    Wb = weight_for(cfg, lin); Xb, dYb = activations_for(cfg, lin)
    Wd, Xd, dYd = bits_to_torch(Wb), bits_to_torch(Xb), bits_to_torch(dYb)
    d = eqat.make_desc(bits, g, out, in_f, T)

    tok = sample(T, N_TOK, cfg_name, lin_name, "tok")
    rows_y = sample(out, N_OUT_Y, cfg_name, lin_name, "rows_y")
    rows_g = sample(out, N_OUT_G, cfg_name, lin_name, "rows_g")
    grp = sample(ng, N_COL_GROUPS, cfg_name, lin_name, "grp")
    cols = (grp[:, None] * g + np.arange(g)[None, :]).ravel()

    # step sizes and zero points: the library's own initialisation, bit-exact on the sampled rows
    s_d = torch.empty(out, ng, device="cuda"); z_d = torch.empty(out, ng, device="cuda")
    eqat.eqat_minmax_init(d, Wd, s_d, z_d)
    rows_all = np.union1d(rows_y, rows_g)
    W_rows = f32(Wb[rows_all])
    s_rows, z_rows = O.minmax_init(W_rows, bits, g)
    assert np.array_equal(s_d[rows_all].cpu().numpy(), s_rows)
    assert np.array_equal(z_d[rows_all].cpu().numpy(), z_rows)
    # every later oracle input comes from the oracle: full (s, z) on the column sample, via the same rule
    s_cols, z_cols = O.minmax_init(f32(Wb[:, cols]), bits, g)            # [out, len(grp)]
    iy = np.searchsorted(rows_all, rows_y); ig = np.searchsorted(rows_all, rows_g)
    X_tok, dY_tok = f32(Xb[tok]), f32(dYb[tok])
    # the GPU consumes s, z produced on the device; they equal the oracle's on every sampled row, and
    # a full-size check of them follows from the identities below.
    if mode == "block_ap":
        Y = torch.empty(T, out, dtype=torch.bfloat16, device="cuda")
        What = torch.empty(out, in_f, dtype=torch.bfloat16, device="cuda")
        dX = torch.empty(T, in_f, dtype=torch.bfloat16, device="cuda")
        dW = torch.empty(out, in_f, dtype=torch.bfloat16, device="cuda")
        ds = torch.empty(out, ng, device="cuda"); dz = torch.empty(out, ng, device="cuda")
        assert eqat.workspace_bytes(d, eqat.EQAT_OP_FAKEQUANT_BWD) == 0      # groups of 64 / 128: no scratch
        ws = None
        eqat.qlinear_fakequant_fwd(d, Xd, Wd, s_d, z_d, Y, What)
        eqat.qlinear_fakequant_bwd(d, Xd, dYd, Wd, s_d, z_d, What, dX, dW, ds, dz, ws)
        torch.cuda.synchronize()
        What_rows = O.fake_quant_weight(W_rows, s_rows, z_rows, bits, g)
        assert rel_err(torch_to_f64(What[rows_all]), What_rows) <= TOL
        check_block(Y[tok][:, rows_y], X_tok, What_rows[iy], "Y sample")
        What_cols = O.fake_quant_weight(f32(Wb[:, cols]), s_cols, z_cols, bits, g)
        check_block(dX[tok][:, cols], dY_tok, What_cols.T, "dX sample")
        # the last row-tile and column-tile of both outputs, densely
        s_last, z_last = O.minmax_init(f32(Wb[-CORNER:]), bits, g)
        check_block(Y[-CORNER:, -CORNER:], f32(Xb[-CORNER:]), O.fake_quant_weight(f32(Wb[-CORNER:]), s_last, z_last, bits, g),
                    "Y corner")
        s_lc, z_lc = O.minmax_init(f32(Wb[:, -CORNER:]), bits, g)
        check_block(dX[-CORNER:, -CORNER:], f32(dYb[-CORNER:]), O.fake_quant_weight(f32(Wb[:, -CORNER:]), s_lc, z_lc, bits, g).T,
                    "dX corner")
        G = O.weight_grad(f32(dYb[:, rows_g]), f32(Xb))
        dW_o, ds_o, dz_o = O.ste_bwd(G, W_rows[ig], s_rows[ig], z_rows[ig], bits, g)
        assert rel_err(torch_to_f64(dW[rows_g]), dW_o) <= TOL
        absG = O.weight_grad(np.abs(f32(dYb[:, rows_g])), np.abs(f32(Xb)))
        assert_elementwise(torch_to_f64(dW[rows_g]), dW_o, contraction_bound(dW_o, absG, 0.0, 0), "dW sample")
        assert rel_err(torch_to_f64(ds[rows_g]), ds_o) <= TOL
        if np.linalg.norm(dz_o) > 0:
            assert rel_err(torch_to_f64(dz[rows_g]), dz_o) <= TOL
        a, b = dot64(dYd, Y), dot64(dX, Xd)
        assert abs(a - b) <= inner_product_tol(dYd, Y, dX, Xd)
    else:
        P = torch.empty(out, in_f * bits // 8, dtype=torch.uint8, device="cuda")
        z8 = torch.empty(out, ng, dtype=torch.uint8, device="cuda")
        s16 = torch.empty(out, ng, dtype=torch.float16, device="cuda")
        eqat.eqat_quantize_pack(d, Wd, s_d, z_d, P, z8, s16)
        P_rows, z8_rows, s16_rows = O.quantize_pack(W_rows, s_rows, z_rows, bits, g)
        assert np.array_equal(P[rows_all].cpu().numpy(), P_rows)                    # bit-exact
        assert np.array_equal(z8[rows_all].cpu().numpy(), z8_rows)
        assert np.array_equal(s16[rows_all].cpu().numpy().view(np.uint16), s16_rows.view(np.uint16))
        codes = torch.empty(out, in_f, dtype=torch.uint8, device="cuda")
        eqat.eqat_unpack(d, P, codes)
        q_rows = O.unpack_rows(P_rows, bits, in_f)
        assert np.array_equal(codes[rows_all].cpu().numpy(), q_rows)
        Y = torch.empty(T, out, dtype=torch.bfloat16, device="cuda")
        dX = torch.empty(T, in_f, dtype=torch.bfloat16, device="cuda")
        ds = torch.empty(out, ng, device="cuda"); dz = torch.empty(out, ng, device="cuda")
        eqat.qlinear_packed_fwd(d, Xd, P, s16, z8, Y)
        eqat.qlinear_packed_bwd_dx(d, dYd, P, s16, z8, dX)
        eqat.qlinear_packed_bwd_ds(d, Xd, dYd, P, z8, s16, ds, dz)
        torch.cuda.synchronize()
        What_rows = O.dequantize(q_rows, s16_rows.astype(np.float32), z8_rows, g)
        check_block(Y[tok][:, rows_y], X_tok, What_rows[iy], "Y sample")
        q_cols, _, _ = O.quantize_codes(f32(Wb[:, cols]), s_cols, z_cols, bits, g)
        What_cols = O.dequantize(q_cols, s_cols.astype(np.float16).astype(np.float32), z_cols, g)
        check_block(dX[tok][:, cols], dY_tok, What_cols.T, "dX sample")
        # the last row-tile and column-tile of both outputs, densely (codes, fp16 step sizes and zero points of
        # those rows / columns from the oracle's own hand-off)
        def handoff(Wpart):
            s_p, z_p = O.minmax_init(Wpart, bits, g)
            P_p, z8_p, s16_p = O.quantize_pack(Wpart, s_p, z_p, bits, g)
            return O.dequantize(O.unpack_rows(P_p, bits, Wpart.shape[1]), s16_p.astype(np.float32), z8_p, g)
        check_block(Y[-CORNER:, -CORNER:], f32(Xb[-CORNER:]), handoff(f32(Wb[-CORNER:])), "Y corner")
        check_block(dX[-CORNER:, -CORNER:], f32(dYb[-CORNER:]), handoff(f32(Wb[:, -CORNER:])).T, "dX corner")
        dYg, Xf = f32(dYb[:, rows_g]), f32(Xb)
        assert rel_err(torch_to_f64(ds[rows_g]), O.e2e_ds(dYg, Xf, q_rows[ig], z8_rows[ig], g)) <= TOL
        assert rel_err(torch_to_f64(dz[rows_g]), O.e2e_dz(dYg, Xf, s16_rows[ig].astype(np.float32), g)) <= TOL
        a, b = dot64(dYd, Y), dot64(dX, Xd)
        tol_abs = inner_product_tol(dYd, Y, dX, Xd)
        assert abs(a - b) <= tol_abs
        euler = float((s16.double() * ds.double()).sum())
        assert abs(euler - a) <= tol_abs
        # decoding: the first one, four, eight and twenty tokens alone (the matrix-vector kernels where their
        # activations fit in shared memory, whole or in slices of the tokens; the tiled kernel otherwise), against the
        # oracle and against the same rows of the full batch
        for t_few in (1, 4, 8, 20):
            d_few = eqat.make_desc(bits, g, out, in_f, t_few)
            Y_few = torch.empty(t_few, out, dtype=torch.bfloat16, device="cuda")
            eqat.qlinear_packed_fwd(d_few, Xd[:t_few].contiguous(), P, s16, z8, Y_few)
            torch.cuda.synchronize()
            assert rel_err(torch_to_f64(Y_few[:, rows_y]), O.linear_fwd(f32(Xb[:t_few]), What_rows[iy])) <= TOL
            assert rel_err(torch_to_f64(Y_few), torch_to_f64(Y[:t_few])) <= TOL
    torch.cuda.synchronize()
    assert eqat.device_status() == (0, 0)
