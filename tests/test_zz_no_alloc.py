"""qlinear_fakequant_bwd_noalloc: the Block-AP backward for callers that cannot
allocate device memory (their device memory belongs to another framework's pool,
or they sit where the synchronisation cudaMalloc may imply is unacceptable).

It must give exactly what qlinear_fakequant_bwd gives with a caller-allocated
workspace (same kernels, same inputs: bit for bit) and what the oracle gives
(within the tolerance of the other parity tests), on two calls in a row (the
built-in scratch array is shared by all calls and keeps the previous call's
contents), and must refuse problems larger than the array.
Collected last so that a failure here cannot mask any other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from helpers import TOL, bits_to_torch, f32, rel_err, torch_to_f64
from oracle import eqat_oracle as O
from workloads import activations_for, get_config, weight_for


@pytest.fixture(scope="module")
def eqat():
    from paper_2407_11062_b200.build import build_library
    build_library()
    from paper_2407_11062_b200 import binding
    return binding


def test_rejects_problems_larger_than_the_builtin_scratch(eqat):
    """Decided on the host before any pointer is touched: needs no GPU."""
    big = eqat.make_desc(2, 64, 4096, 4096, 256)                 # 16 Mi elements > 4 Mi
    assert big.out_features * big.in_features > eqat.NOALLOC_MAX_WEIGHT_ELEMS
    fake = ctypes.c_void_p(0x1000)
    rc = eqat.lib.qlinear_fakequant_bwd_noalloc(ctypes.byref(big), *([fake] * 10), None)
    assert rc == eqat.EQAT_ERR_WORKSPACE
    assert eqat.lib.qlinear_fakequant_bwd_noalloc(None, *([fake] * 10), None) == eqat.EQAT_ERR_NULL


@pytest.mark.gpu
@pytest.mark.parametrize("channel_wise", [True, False])
def test_matches_the_workspace_variant_twice_in_a_row(eqat, channel_wise):
    """Channel-wise groups are the case that uses the scratch (a group longer than an output tile sends the
    gradient of W_hat through memory); the short-group case checks that the entry point agrees there too."""
    cfg = get_config("c1"); lin = cfg.linears[0]
    out, in_f, T, bits = lin.out_features, lin.in_features, cfg.tokens, cfg.bits
    g = in_f if channel_wise else cfg.group
    ng = in_f // g
    Wb = weight_for(cfg, lin); Xb, dYb = activations_for(cfg, lin)
    s, z = O.minmax_init(f32(Wb), bits, g)
    s = (s * np.float32(0.8)).astype(np.float32)                 # clamps on both sides: dz is not all zero
    Wd, Xd, sd, zd = bits_to_torch(Wb), bits_to_torch(Xb), torch.from_numpy(s).cuda(), torch.from_numpy(z).cuda()
    d = eqat.make_desc(bits, g, out, in_f, T)
    Y = torch.empty(T, out, dtype=torch.bfloat16, device="cuda")
    What = torch.empty(out, in_f, dtype=torch.bfloat16, device="cuda")
    eqat.qlinear_fakequant_fwd(d, Xd, Wd, sd, zd, Y, What)

    def outputs():
        return (torch.empty(T, in_f, dtype=torch.bfloat16, device="cuda"),
                torch.empty(out, in_f, dtype=torch.bfloat16, device="cuda"),
                torch.empty(out, ng, device="cuda"), torch.empty(out, ng, device="cuda"))

    # two different upstream gradients, so the second call must not see the first call's scratch
    dY1 = bits_to_torch(dYb)
    dY2 = (dY1.float() * -0.5 + 0.003).to(torch.bfloat16)
    n_ws = eqat.workspace_bytes(d, eqat.EQAT_OP_FAKEQUANT_BWD)
    assert (n_ws > 0) == channel_wise
    ws = torch.empty(n_ws, dtype=torch.uint8, device="cuda") if n_ws else None
    W32, X32 = f32(Wb), f32(Xb)
    What_o = O.fake_quant_weight(W32, s, z, bits, g)
    for dY in (dY1, dY2):
        ref = outputs(); got = outputs()
        eqat.qlinear_fakequant_bwd(d, Xd, dY, Wd, sd, zd, What, *ref, ws)
        eqat.qlinear_fakequant_bwd_noalloc(d, Xd, dY, Wd, sd, zd, What, *got)
        torch.cuda.synchronize()
        for name, a, b in zip(("dX", "dW", "ds", "dz"), got, ref):
            assert np.linalg.norm(torch_to_f64(b)) > 0, name
            assert torch.equal(a, b), name                       # the same kernels on the same inputs
        # and against the oracle (Eqs. 3-5 on the fp64 weight gradient)
        dY64 = torch_to_f64(dY)
        dW_o, ds_o, dz_o = O.ste_bwd(O.weight_grad(dY64, X32), W32, s, z, bits, g)
        for name, a, b in zip(("dX", "dW", "ds", "dz"), got, (O.linear_bwd_dx(dY64, What_o), dW_o, ds_o, dz_o)):
            assert rel_err(torch_to_f64(a), b) <= TOL, name
    assert eqat.device_status() == (0, 0)
