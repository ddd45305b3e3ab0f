"""Shared helpers of the tests: bf16 bit patterns <-> torch / numpy, error norms."""
import numpy as np
import torch

from workloads import from_bf16_bits, to_bf16_bits

TOL = 5e-3          # relative Frobenius error allowed on floating-point outputs


def bits_to_torch(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor on `device` (same bytes)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.to(device)


def torch_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def rel_err(a, b) -> float:
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    nb = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / nb) if nb > 0 else float(np.linalg.norm(a))


def f32(bits):
    return from_bf16_bits(bits)


def bf16_round(x):
    return from_bf16_bits(to_bf16_bits(np.asarray(x, np.float32)))


# --------------------------------------------------------------------------- guard words
GUARD_BYTES = 256
_SENTINEL = 0xA5


class Guarded:
    """Output buffers carved out of sentinel-filled allocations, 256 bytes of guard on each side.

    The sanitizer is not available where these tests run, so this is how a store that lands before or past
    an output (a ragged last tile, a vector store across the end of a row) shows up: `check()` fails if any
    guard byte changed.  The payload itself starts as sentinel bytes too, so an element the kernel never
    wrote is not mistaken for a result either (0xA5A5 is a large negative bf16, 0xA5A5A5A5 a tiny float).
    """

    def __init__(self):
        self._bufs = []

    def empty(self, *shape, dtype=torch.float32, device="cuda", shift_bytes=0):
        """A contiguous tensor of `shape`; `shift_bytes` (a multiple of 16) moves it off 32/64/... byte boundaries."""
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        assert shift_bytes % 16 == 0 and 0 <= shift_bytes < GUARD_BYTES
        raw = torch.full((GUARD_BYTES + shift_bytes + n + GUARD_BYTES,), _SENTINEL, dtype=torch.uint8, device=device)
        assert raw.data_ptr() % 256 == 0
        view = raw[GUARD_BYTES + shift_bytes: GUARD_BYTES + shift_bytes + n].view(dtype).view(*shape)
        self._bufs.append((raw, GUARD_BYTES + shift_bytes, n))
        return view

    def check(self):
        torch.cuda.synchronize()
        for i, (raw, lo, n) in enumerate(self._bufs):
            assert bool((raw[:lo] == _SENTINEL).all()), f"guard before output {i} was overwritten"
            assert bool((raw[lo + n:] == _SENTINEL).all()), f"guard after output {i} was overwritten"


# --------------------------------------------------------------------------- element-wise bounds
BF16_U = 2.0 ** -8          # unit roundoff of bf16 (8 significant bits): |rn(x) - x| <= 2^-8 |x|


def contraction_bound(ref, abs_terms, sq_terms, operand_roundings=1):
    """How far one element of a bf16 x bf16 -> fp32 contraction, rounded to bf16, may sit from the exact
    value `ref` when the kernel is right.  Three sources:
      * the final rounding to bf16: at most 2^-8 |ref| (and as much again on the error the sum carries,
        covered by the factor 1.05);
      * `operand_roundings` operands that the kernel rounds to bf16 while the reference keeps them exact (the
        fake-quantised / dequantised weight): term k moves by d_k a_k b_k with |d_k| <= 2^-8.  The other
        operand is zero-mean noise here, so these add like a random walk: standard deviation at most
        2^-8 sqrt(sum_k a_k^2 b_k^2); eight of them are allowed (a miss has probability ~1e-15 per element,
        and the inputs are seeded, so a passing case passes for good);
      * fp32 accumulation inside the tensor core and across K blocks, in any order and whether it rounds or
        truncates: 2^-16 sum_k |a_k b_k| is 256 units in the last place of the largest partial sum.
    `abs_terms` = sum_k |a_k| |b_k| and `sq_terms` = sum_k a_k^2 b_k^2 come from the oracle's own contraction
    of |A|, |B| and of A^2, B^2.  For the shapes tested the bound is a few percent of a typical element:
    a 16-byte piece written to the wrong place, or never written, is far outside it."""
    walk = 8.0 * operand_roundings * BF16_U * np.sqrt(sq_terms)
    return (BF16_U * np.abs(ref) + walk + 2.0 ** -16 * abs_terms) * 1.05 + 1e-30


def assert_elementwise(got, ref, bound, what):
    got = np.asarray(got, np.float64)
    err = np.abs(got - ref)
    bad = np.argwhere(~(err <= bound))
    assert bad.size == 0, (what, len(bad), bad[:4].tolist(),
                           [(float(got[tuple(i)]), float(ref[tuple(i)]), float(bound[tuple(i)])) for i in bad[:4]])
