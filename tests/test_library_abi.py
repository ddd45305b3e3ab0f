"""The shared library loads without a GPU, exports every symbol the header
declares, and rejects bad arguments on the host before launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def eqat():
    from paper_2407_11062_b200.build import build_library
    build_library()
    from paper_2407_11062_b200 import binding
    return binding


def _declared():
    src = open(os.path.join(ROOT, "include", "eqat.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b((?:eqat|qlinear)_[a-z0-9_]+)\s*\(", src)))


def test_every_declared_symbol_is_exported(eqat):
    names = _declared()
    assert len(names) >= 17
    raw = ctypes.CDLL(eqat.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n
        assert hasattr(eqat, n) or hasattr(eqat.lib, n)


def test_status_strings(eqat):
    assert eqat.status_string(0) == "ok"
    seen = {eqat.status_string(s) for s in range(-7, 1)}
    assert len(seen) == 8
    assert eqat.lib.eqat_version() >= 100


def test_workspace_sizes(eqat):
    d = eqat.make_desc(2, 64, 512, 512, 256)
    assert eqat.workspace_bytes(d, eqat.EQAT_OP_FAKEQUANT_BWD) == 0          # reduced inside the GEMM: no scratch
    assert eqat.workspace_bytes(eqat.make_desc(2, 256, 512, 512, 256), eqat.EQAT_OP_FAKEQUANT_BWD) == 0
    dc = eqat.make_desc(2, 512, 512, 512, 256)                               # channel-wise: dW_hat in bf16
    assert eqat.workspace_bytes(dc, eqat.EQAT_OP_FAKEQUANT_BWD) == 512 * 512 * 2
    assert eqat.workspace_bytes(d, eqat.EQAT_OP_PACKED_BWD_DS) == 0
    with pytest.raises(eqat.EqatError):
        eqat.workspace_bytes(d, 99)


@pytest.mark.parametrize("kw,status", [
    (dict(bits=5), -4), (dict(bits=1), -4), (dict(group=48), -2), (dict(group=96), -2), (dict(in_features=500), -2),
    (dict(out_features=0), -2), (dict(dz_mode=2), -4), (dict(group=1024), -2),
])
def test_bad_descriptors_are_rejected_on_the_host(eqat, kw, status):
    base = dict(bits=2, group=64, out_features=512, in_features=512, tokens=256, dz_mode=0)
    base.update(kw)
    d = eqat.make_desc(**base)
    fake = ctypes.c_void_p(0x1000)       # never dereferenced: validation fails first
    rc = eqat.lib.eqat_fakequant_weight(ctypes.byref(d), fake, fake, fake, fake, None)
    assert rc == status


def test_null_and_misaligned_pointers(eqat):
    d = eqat.make_desc(2, 64, 512, 512, 256)
    ok, odd = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1004)
    assert eqat.lib.eqat_fakequant_weight(ctypes.byref(d), ok, ok, None, ok, None) == eqat.EQAT_ERR_NULL
    assert eqat.lib.eqat_fakequant_weight(ctypes.byref(d), ok, odd, ok, ok, None) == eqat.EQAT_ERR_ALIGN
    assert eqat.lib.eqat_fakequant_weight(None, ok, ok, ok, ok, None) == eqat.EQAT_ERR_NULL
    assert eqat.lib.qlinear_packed_fwd(ctypes.byref(d), ok, ok, ok, ok, None, None) == eqat.EQAT_ERR_NULL
    # packed GEMMs: a group longer than 256 must be the whole row; GEMMs need tokens > 0 and out % 64 == 0
    d512 = eqat.make_desc(2, 512, 512, 1024, 256)
    assert eqat.lib.qlinear_packed_fwd(ctypes.byref(d512), ok, ok, ok, ok, ok, None) == eqat.EQAT_ERR_UNSUPPORTED
    # zero-point formats: fp16 zero points exist for the packed entry points only; unknown formats nowhere
    dz16 = eqat.make_desc(2, 64, 512, 512, 256, 0, eqat.EQAT_ZP_FP16)
    assert eqat.lib.eqat_fakequant_weight(ctypes.byref(dz16), ok, ok, ok, ok, None) == eqat.EQAT_ERR_UNSUPPORTED
    assert eqat.lib.qlinear_fakequant_fwd(ctypes.byref(dz16), ok, ok, ok, ok, ok, ok, None) == eqat.EQAT_ERR_UNSUPPORTED
    assert eqat.lib.qlinear_packed_fwd(ctypes.byref(dz16), ok, ok, ok, None, ok, None) == eqat.EQAT_ERR_NULL
    dz9 = eqat.make_desc(2, 64, 512, 512, 256, 0, 9)
    assert eqat.lib.qlinear_packed_fwd(ctypes.byref(dz9), ok, ok, ok, ok, ok, None) == eqat.EQAT_ERR_UNSUPPORTED
    # one group per row: the step-size gradient needs scratch for the per-tile sums
    dcw = eqat.make_desc(2, 1024, 512, 1024, 256)
    assert eqat.workspace_bytes(dcw, eqat.EQAT_OP_PACKED_BWD_DS) == 2 * 4 * 512 * 4
    assert eqat.lib.qlinear_packed_bwd_ds(ctypes.byref(dcw), ok, ok, ok, ok, ok, ok, None, None, 0, None) == eqat.EQAT_ERR_WORKSPACE
    d0 = eqat.make_desc(2, 64, 512, 512, 0)
    assert eqat.lib.qlinear_packed_fwd(ctypes.byref(d0), ok, ok, ok, ok, ok, None) == eqat.EQAT_ERR_SHAPE
    d96 = eqat.make_desc(2, 64, 96, 512, 256)
    assert eqat.lib.qlinear_fakequant_fwd(ctypes.byref(d96), ok, ok, ok, ok, ok, ok, None) == eqat.EQAT_ERR_SHAPE
    # workspace of the channel-wise backward: missing, too small, misaligned
    dc = eqat.make_desc(2, 512, 512, 512, 256)
    args = [ok] * 10
    assert eqat.lib.qlinear_fakequant_bwd(ctypes.byref(dc), *args, None, 0, None) == eqat.EQAT_ERR_WORKSPACE
    assert eqat.lib.qlinear_fakequant_bwd(ctypes.byref(dc), *args, ok, 16, None) == eqat.EQAT_ERR_WORKSPACE
    assert eqat.lib.qlinear_fakequant_bwd(ctypes.byref(dc), *args, ctypes.c_void_p(0x1010), 1 << 20, None) == eqat.EQAT_ERR_WORKSPACE
    assert eqat.lib.eqat_selftest_wait_expiry(7, None) == eqat.EQAT_ERR_UNSUPPORTED


def test_block_level_calls_validate_every_linear_before_anything_runs(eqat):
    """eqat_block_ap_step / eqat_e2e_qp_step: a fault in the LAST linear of the array is reported with its index and
    with the status the layer entry point would give; the pointers of the earlier (valid) linears are fake, so a
    launch on them before the check of the last one would not go unnoticed on a machine with a GPU, and on this
    one no launch is possible at all."""
    ok = 0x1000
    d = eqat.make_desc(2, 64, 512, 512, 256)

    def ap(**kw):
        f = dict(desc=d, X=ok, dY=ok, W=ok, s=ok, z=ok, Y=ok, W_hat=ok, dX=ok, dW=ok, ds=ok, dz=ok, workspace=None,
                 workspace_bytes=0)
        f.update(kw)
        return eqat.eqat_block_ap_linear(**f)

    def e2e(**kw):
        f = dict(desc=d, X=ok, dY=ok, Wq_packed=ok, s16=ok, z=ok, Y=ok, dX=ok, ds=ok, dz=None, workspace=None,
                 workspace_bytes=0)
        f.update(kw)
        return eqat.eqat_e2e_qp_linear(**f)

    failed = ctypes.c_int(-5)
    for rows, fn, struct, want in (
            ([ap(), ap(), ap(dW=None)], eqat.lib.eqat_block_ap_step, eqat.eqat_block_ap_linear, (eqat.EQAT_ERR_NULL, 2)),
            ([ap(), ap(Y=0x1004)], eqat.lib.eqat_block_ap_step, eqat.eqat_block_ap_linear, (eqat.EQAT_ERR_ALIGN, 1)),
            ([ap(), ap(desc=eqat.make_desc(2, 512, 512, 512, 256))], eqat.lib.eqat_block_ap_step,
             eqat.eqat_block_ap_linear, (eqat.EQAT_ERR_WORKSPACE, 1)),              # channel-wise without scratch
            ([e2e(), e2e(), e2e(), e2e(ds=None)], eqat.lib.eqat_e2e_qp_step, eqat.eqat_e2e_qp_linear,
             (eqat.EQAT_ERR_NULL, 3)),
            ([e2e(), e2e(desc=eqat.make_desc(5, 64, 512, 512, 256))], eqat.lib.eqat_e2e_qp_step,
             eqat.eqat_e2e_qp_linear, (eqat.EQAT_ERR_UNSUPPORTED, 1)),
            ([e2e(), e2e(dz=ok, s16=None)], eqat.lib.eqat_e2e_qp_step, eqat.eqat_e2e_qp_linear, (eqat.EQAT_ERR_NULL, 1))):
        arr = (struct * len(rows))(*rows)
        rc = fn(arr, len(rows), ctypes.byref(failed), None)
        assert (rc, failed.value) == want
    assert eqat.lib.eqat_block_ap_step(None, 1, None, None) == eqat.EQAT_ERR_NULL
    arr = (eqat.eqat_e2e_qp_linear * 1)(e2e())
    assert eqat.lib.eqat_e2e_qp_step(arr, 0, None, None) == eqat.EQAT_ERR_SHAPE
