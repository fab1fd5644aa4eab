"""Helpers shared by the GPU parity tests (comparison rules, code unpacking)."""
import numpy as np
import torch

from oracle import oracle as O

# Tolerances, from the arithmetic:
#  * integer accumulators and codes of bit-identical inputs: exact;
#  * fp32 gate / cell / log-prob values: the GPU evaluates in fp32 what the oracle evaluates
#    in double, a handful of roundings at 2^-24 relative on values of magnitude <= ~10 plus a
#    2-ulp expf/tanhf: 1e-5 relative with a 2e-6 absolute floor;
#  * a code made from such a float can differ by one step only where the float sits within
#    1e-3 code units of a rounding tie (the fp32 error times inv_scale <= 127 is ~1e-4).
RTOL, ATOL, TIE = 1e-5, 2e-6, 1e-3


def gpu_codes(t: torch.Tensor, k: int, act) -> np.ndarray:
    """Packed device codes [rows, bytes] -> int16 [rows, k]."""
    b = t.detach().cpu().numpy()
    b = b.reshape(-1, b.shape[-1])
    if act.bits == 4:
        return O.unpack4(b, k, bool(act.is_signed))
    return b.view(np.int8)[:, :k].astype(np.int16)


def pack_codes(q: np.ndarray, act, k_pad=None) -> torch.Tensor:
    """Oracle codes [rows, k] -> device tensor in the library's storage format."""
    q = np.ascontiguousarray(q, dtype=np.int16)
    rows, k = q.shape
    k_pad = k_pad or (k + 31) // 32 * 32
    pad = 0 if act.is_signed else act.zero_point
    if act.bits == 4:
        b = O.pack4(q, k_pad, pad)
    else:
        b = np.zeros((rows, k_pad), dtype=np.int8)
        b[:, :k] = q.astype(np.int8)
        b = b.view(np.uint8)
    return torch.from_numpy(b).cuda()


def near_tie(h: np.ndarray, act) -> np.ndarray:
    v = h.astype(np.float64) * act.inv_scale
    return np.abs(v - np.floor(v) - 0.5) < TIE


def assert_codes_match(got: np.ndarray, want: np.ndarray, h_oracle: np.ndarray, act, what=""):
    """Bit-exact except where the oracle's float is a near-tie (then +-1 code is accepted)."""
    diff = got.astype(np.int32) - want.astype(np.int32)
    bad = diff != 0
    if not bad.any():
        return 0
    tie = near_tie(h_oracle, act)
    outside = bad & ~(tie & (np.abs(diff) <= 1))
    assert not outside.any(), f"{what}: {outside.sum()} code mismatches outside near-ties " \
                              f"(of {bad.sum()} mismatches, {got.size} codes)"
    return int(bad.sum())


def assert_close(got, want, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    err = np.abs(got - want)
    tol = ATOL + RTOL * np.abs(want)
    assert (err <= tol).all(), f"{what}: max err {err.max():.3e} (worst excess {(err - tol).max():.3e})"


def to_act(a):
    """oracle Act -> library Act (same five constants)."""
    from paper_2206_07882_b200 import binding as Bd
    return Bd.Act(a.scale, a.inv_scale, a.zero_point, a.bits, a.is_signed)
