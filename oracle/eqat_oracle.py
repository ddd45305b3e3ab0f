"""CPU oracle for the group-wise low-bit quantised linear layer of EfficientQAT.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  Nothing in the product package imports it and
it imports nothing from the product package; it shares no code, table or helper
with the CUDA path.  Only the tests, the smoke check and the CPU-baseline leg of
the benchmark may call it.

Every function is the paper's definition written out with numpy, one element at
a time in effect (vectorised over the array, never blocked, fused or
reordered).  Every sum is accumulated in float64.  The one place where float32
is used on purpose is the quotient w/s that decides the integer code (see
``quantize_codes``): a code is a discontinuous function of that quotient, so
the precision in which the decision is taken is part of the definition.

Conventions (paper Sec. 3.2 gives the maths; the tensor layout is this
library's): ``W[out, in]`` row-major as in ``Y = X @ W.T``; a quantisation group
is a run of ``group`` consecutive elements along ``in`` inside one row; ``s`` and
``z`` have shape ``[out, in // group]``; ``Q = 2**bits - 1``.

Pins (tests/test_oracle_pins.py): hand-worked one-group example of Eqs. 1-5,
finite differences of Eq. 2 on the clamped branches and of the STE surrogate on
the in-range branch, idempotence and grid membership of the quantiser, textbook
triple-loop matmuls and adjoint identities for the three contractions,
brute-force group sums and exact finite differences for the E2E-QP step-size
gradient, exhaustive round trips, hand-evaluated byte patterns and the paper's
bits-per-parameter table for the codec, hand-derived FP16 bit patterns and
clamped N-bit zero points for the side outputs of the hand-off.

Parity unpinned by the paper (conventions of this library, each exercised by a
test but fixed by no printed value): the bit layout of the packed stream, the
tie-break of the rounding (half to even), and rounding a fractional zero point
before use.
"""
from __future__ import annotations

import numpy as np

FP16_MIN_NORMAL = np.float32(2.0 ** -14)


def qmax(bits: int) -> int:
    """Largest code of an N-bit quantiser, 2^N - 1 (Eq. 1)."""
    return (1 << int(bits)) - 1


def _per_element(p: np.ndarray, group: int) -> np.ndarray:
    """Broadcast a per-group array [out, in/group] to per-element [out, in]."""
    return np.repeat(p, group, axis=1)


def _check(W, s, group):
    out, in_f = W.shape
    if in_f % group:
        raise ValueError("in_features must be a multiple of group")
    if s.shape != (out, in_f // group):
        raise ValueError("s/z must have shape [out, in/group]")


def round_zero_point(z: np.ndarray) -> np.ndarray:
    """Zero point as used by Eq. 1: the nearest integer (ties to even).

    The paper stores z in N bits (Sec. 3.2, last paragraph) while training it
    as a real number; this library reads that as "the forward pass sees rint(z)
    and the gradient passes straight through".  Integer-valued z is unchanged.
    """
    return np.rint(np.asarray(z, np.float32)).astype(np.float64)


def quantize_codes(W, s, z, bits: int, group: int):
    """Eq. 1:  W_int = clamp(round(W / s) + z, 0, 2^N - 1).

    Returns ``(q, r, p)``: the integer codes (int32), the rounded quotient
    round(W/s) and the pre-clamp value round(W/s) + z (both float64, integer
    valued).  The quotient is formed in IEEE binary32 with round-to-nearest-even
    from the float32 values of ``W`` and ``s`` and rounded with ties to even.
    """
    W32 = np.ascontiguousarray(W, np.float32)
    s32 = np.ascontiguousarray(s, np.float32)
    _check(W32, s32, group)
    t = W32 / _per_element(s32, group)            # binary32 division
    r = np.rint(t).astype(np.float64)             # ties to even
    p = r + _per_element(round_zero_point(z), group)
    q = np.clip(p, 0.0, float(qmax(bits))).astype(np.int32)
    return q, r, p


def _zero_point(z, real_zero_point: bool) -> np.ndarray:
    """The zero point Eq. 2 subtracts.  In Block-AP and in E2E-QP with frozen zero points it is the integer that is
    stored in N bits (``round_zero_point``).  The E2E-QP variants that train z (Sec. 3.3 and the table of E2E-QP
    trainable parameters, where z is promoted to FP16: 2.50 average bits at w2g64) run no quantiser, only Eq. 2, so
    their z enters as the real number it is: ``real_zero_point=True`` takes it unrounded."""
    return np.asarray(z, np.float64) if real_zero_point else round_zero_point(z)


def dequantize(q, s, z, group: int, real_zero_point: bool = False) -> np.ndarray:
    """Eq. 2:  W_hat = (W_int - z) * s, in float64."""
    q64 = np.asarray(q, np.float64)
    s64 = _per_element(np.asarray(s, np.float64), group)
    z64 = _per_element(_zero_point(z, real_zero_point), group)
    return (q64 - z64) * s64


def fake_quant_weight(W, s, z, bits: int, group: int) -> np.ndarray:
    """Eq. 2 applied to Eq. 1: the weight the Block-AP forward pass multiplies by."""
    q, _, _ = quantize_codes(W, s, z, bits, group)
    return dequantize(q, s, z, group)


def linear_fwd(X, W_hat) -> np.ndarray:
    """Y[t, o] = sum_j X[t, j] * W_hat[o, j]   (forward of the linear layer)."""
    return np.asarray(X, np.float64) @ np.asarray(W_hat, np.float64).T


def linear_bwd_dx(dY, W_hat) -> np.ndarray:
    """dX[t, j] = sum_o dY[t, o] * W_hat[o, j]   (chain rule through Y = X W_hat^T)."""
    return np.asarray(dY, np.float64) @ np.asarray(W_hat, np.float64)


def weight_grad(dY, X) -> np.ndarray:
    """G[o, j] = sum_t dY[t, o] * X[t, j]   (gradient of the loss w.r.t. W_hat)."""
    return np.asarray(dY, np.float64).T @ np.asarray(X, np.float64)


def ste_partials(W, s, z, bits: int, group: int, dz_mode: int = 0):
    """Per-element partial derivatives of W_hat (Appendix "Gradient of
    Trainable Parameters in Block-AP", Eqs. 3-5), with the upper bound read as
    2^N - 1 as in Eq. 1 and both bounds inclusive as printed.

    Returns ``(dw_dw, dw_ds, dw_dz)`` as float64 arrays [out, in]:
      in range (0 <= round(w/s)+z <= Q):  1,  round(w/s) - w/s,  0
      below    (round(w/s)+z < 0):        0,  -z,                -s  (or -1)
      above    (round(w/s)+z > Q):        0,  Q - z,             -s  (or -1)
    ``dz_mode`` 0 gives the clamped-branch value -s that differentiating Eq. 2
    with a saturated code yields; 1 gives the literal -1 printed in Eq. 4.
    """
    Q = float(qmax(bits))
    _, r, p = quantize_codes(W, s, z, bits, group)
    s64 = _per_element(np.asarray(s, np.float64), group)
    z64 = _per_element(round_zero_point(z), group)
    frac = r - np.asarray(W, np.float64) / s64     # round(w/s) - w/s
    below = p < 0.0
    above = p > Q
    inside = ~(below | above)
    dw_dw = inside.astype(np.float64)
    dw_ds = np.where(inside, frac, np.where(below, -z64, Q - z64))
    clamp_dz = -s64 if dz_mode == 0 else -np.ones_like(s64)
    dw_dz = np.where(inside, 0.0, clamp_dz)
    return dw_dw, dw_ds, dw_dz


def _group_sum(A: np.ndarray, group: int) -> np.ndarray:
    out, in_f = A.shape
    return A.reshape(out, in_f // group, group).sum(axis=2, dtype=np.float64)


def ste_bwd(G, W, s, z, bits: int, group: int, dz_mode: int = 0):
    """Block-AP backward through the fake quantiser (Eqs. 3-5 and the chain
    rule): given G = dL/dW_hat returns ``(dW, ds, dz)`` with
    dW = G * dW_hat/dw, ds[o,g] = sum_{j in g} G * dW_hat/ds,
    dz[o,g] = sum_{j in g} G * dW_hat/dz."""
    G64 = np.asarray(G, np.float64)
    dw_dw, dw_ds, dw_dz = ste_partials(W, s, z, bits, group, dz_mode)
    return G64 * dw_dw, _group_sum(G64 * dw_ds, group), _group_sum(G64 * dw_dz, group)


def e2e_ds(dY, X, q, z, group: int, real_zero_point: bool = False) -> np.ndarray:
    """E2E-QP step-size gradient (Sec. 3.3: d w_hat / d s = w_q - z):
    ds[o,g] = sum_{j in g} (sum_t dY[t,o] X[t,j]) * (q[o,j] - z[o,g]).
    The full weight gradient is materialised first, then multiplied and summed."""
    G = weight_grad(dY, X)
    z64 = _per_element(_zero_point(z, real_zero_point), group)
    return _group_sum(G * (np.asarray(q, np.float64) - z64), group)


def e2e_dz(dY, X, s, group: int) -> np.ndarray:
    """E2E-QP zero-point gradient when z is trained (Sec. 3.3 variant): from
    Eq. 2, d w_hat / d z = -s, so dz[o,g] = -s[o,g] * sum_{j in g} G[o,j]."""
    G = weight_grad(dY, X)
    return -np.asarray(s, np.float64) * _group_sum(G, group)


def minmax_init(W, bits: int, group: int):
    """Round-to-nearest initialisation of (s, z) from each group's range:
    s = (max - min) / Q, z = -round(min / s), both in binary32.  The paper does
    not describe the initialisation; this is the usual min/max rule.  Two
    guards keep the result storable in the paper's format (fp16 step size,
    N-bit zero point): s is raised to the smallest normal fp16 and z is clamped
    to [0, Q]."""
    W32 = np.ascontiguousarray(W, np.float32)
    out, in_f = W32.shape
    Wg = W32.reshape(out, in_f // group, group)
    mx = Wg.max(axis=2)
    mn = Wg.min(axis=2)
    Qf = np.float32(qmax(bits))
    s = ((mx - mn) / Qf).astype(np.float32)
    s = np.maximum(s, FP16_MIN_NORMAL)
    z = -np.rint(mn / s)
    z = np.clip(z, np.float32(0), Qf).astype(np.float32)
    return s, z + np.float32(0.0)   # +0.0 turns -0.0 into +0.0


# ---------------------------------------------------------------------------
# Storage format.  The paper gives sizes only (N-bit codes and zero points,
# fp16 step sizes, N + (N+16)/g bits per parameter); the bit order below is this
# library's: a dense little-endian bit stream.
# ---------------------------------------------------------------------------

def pack_stream(codes, bits: int) -> np.ndarray:
    """Pack a 1-D array of N-bit codes into bytes: code j occupies stream bits
    [N*j, N*j + N); stream bit b is bit (b % 8) of byte (b // 8)."""
    c = np.asarray(codes).astype(np.uint8).ravel()
    if (c.size * bits) % 8:
        raise ValueError("stream does not end on a byte boundary")
    bitplanes = (c[:, None] >> np.arange(bits, dtype=np.uint8)[None, :]) & 1   # [n, N] LSB first
    return np.packbits(bitplanes.ravel().astype(np.uint8), bitorder="little")


def unpack_stream(packed, bits: int, count: int) -> np.ndarray:
    b = np.unpackbits(np.asarray(packed, np.uint8).ravel(), bitorder="little")[: count * bits]
    b = b.reshape(count, bits).astype(np.uint32)
    return (b << np.arange(bits, dtype=np.uint32)[None, :]).sum(axis=1).astype(np.uint8)


def pack_rows(codes, bits: int) -> np.ndarray:
    """Pack codes[out, in] row by row: each row is its own bit stream of
    in*N/8 bytes (rows start on byte boundaries)."""
    c = np.asarray(codes)
    out, in_f = c.shape
    if (in_f * bits) % 8:
        raise ValueError("row does not end on a byte boundary")
    return np.stack([pack_stream(c[o], bits) for o in range(out)], axis=0)


def unpack_rows(packed, bits: int, in_features: int) -> np.ndarray:
    p = np.asarray(packed, np.uint8)
    return np.stack([unpack_stream(p[o], bits, in_features) for o in range(p.shape[0])], axis=0)


def quantize_pack(W, s, z, bits: int, group: int):
    """Hand-off from Block-AP to E2E-QP (Sec. 3.2 last paragraph, Sec. 3.3):
    codes of Eq. 1 packed to N bits, zero points as small integers, step sizes
    rounded to fp16.  Returns ``(packed[out, in*N/8] uint8, z8[out, in/g] uint8,
    s16[out, in/g] float16)``."""
    q, _, _ = quantize_codes(W, s, z, bits, group)
    z8 = np.clip(round_zero_point(z), 0, qmax(bits)).astype(np.uint8)
    s16 = np.asarray(s, np.float32).astype(np.float16)
    return pack_rows(q, bits), z8, s16


def packed_bytes(out_features: int, in_features: int, bits: int, group: int) -> int:
    """Stored size of one quantised linear: N-bit codes, N-bit zero points
    (one flat stream), fp16 step sizes."""
    n = out_features * in_features
    ng = n // group
    return n * bits // 8 + (ng * bits + 7) // 8 + 2 * ng
