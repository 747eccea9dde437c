"""CPU oracle of the TopLoc proof path (ctypes view of oracle/toploc_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The product package never imports this module
and this module never imports the product package.

All functions take and return numpy arrays on the host.
"""
import ctypes
import os

import numpy as np

from . import build as _build

P_FIELD = 65521          # largest prime below 2^16 (Algorithm 3 needs a prime that fits 2 bytes)
M_HIGH = 65536           # Algorithm 6 search range, inclusive
M_LOW = 2 ** 15 + 1
Q_FIELD = 2 ** 32 - 5    # 32-bit field variant: largest prime below 2^32 (fits 4-byte coefficients)

ST_OK, ST_NO_MODULUS, ST_K_EXCEEDS, ST_BAD_PROOF, ST_NONFINITE = range(5)

RESULT_DTYPE = np.dtype([
    ("exp_mismatch", "<u4"), ("n_match", "<u4"), ("mant_diff_sum", "<u4"), ("topk_mismatch", "<i4"),
    ("mant_mean", "<f8"), ("mant_median", "<f8"), ("modulus", "<u4"),
    ("accept", "u1"), ("status", "u1"), ("pad", "u1", (2,)),
])
assert RESULT_DTYPE.itemsize == 40

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        _lib.oracle_find_injective_modulus.restype = ctypes.c_uint32
        _lib.oracle_mod_inverse.restype = ctypes.c_uint32
        _lib.oracle_mod_inverse_euclid.restype = ctypes.c_int64
        _lib.oracle_horner.restype = ctypes.c_uint32
        _lib.oracle_num_chunks.restype = ctypes.c_int64
        _lib.oracle_mod_inverse32.restype = ctypes.c_uint32
        _lib.oracle_horner32.restype = ctypes.c_uint32
    return _lib


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _dtype_code(act):
    """bf16 chunks travel as uint16 bit patterns, fp32 chunks as float32 or uint32."""
    if act.dtype == np.uint16:
        return 0
    if act.dtype in (np.float32, np.uint32):
        return 1
    raise TypeError("activations must be uint16 (bf16 patterns), float32 or uint32")


def default_threads():
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def topk(chunk, k):
    """chunk: 2-D [rows, hidden] array -> (indices uint32[k], bits uint16[k]) in rank order,
    or None when k exceeds the chunk."""
    chunk = np.ascontiguousarray(chunk)
    rows, hidden = chunk.shape
    idx = np.zeros(k, np.uint32)
    bits = np.zeros(k, np.uint16)
    st = lib().oracle_topk(_ptr(chunk), _dtype_code(chunk), rows, hidden, ctypes.c_int64(hidden), k,
                           _ptr(idx), _ptr(bits))
    return None if st != ST_OK else (idx, bits)


def find_injective_modulus(indices, field_distinct=True):
    """Algorithm 6; returns 0 when there is none."""
    idx = np.ascontiguousarray(indices, np.uint32)
    return int(lib().oracle_find_injective_modulus(_ptr(idx), len(idx), int(bool(field_distinct))))


def mod_inverse(a):
    return int(lib().oracle_mod_inverse(ctypes.c_uint32(a)))


def mod_inverse_euclid(a, m):
    return int(lib().oracle_mod_inverse_euclid(ctypes.c_int64(a), ctypes.c_int64(m)))


def interpolate(x, y, lagrange=False):
    """Coefficients (ascending degree, uint16) of the polynomial through (x_j, y_j) over Z_p:
    by elimination on the Vandermonde system, or (the second statement) by Lagrange's form."""
    x = np.ascontiguousarray(x, np.uint32)
    y = np.ascontiguousarray(y, np.uint32)
    c = np.zeros(len(x), np.uint16)
    fn = lib().oracle_interpolate_lagrange if lagrange else lib().oracle_interpolate
    if fn(_ptr(x), _ptr(y), len(x), _ptr(c)) != 0:
        raise ValueError("x values are not distinct mod p")
    return c


def horner(coeffs, x):
    c = np.ascontiguousarray(coeffs, np.uint16)
    return int(lib().oracle_horner(_ptr(c), len(c), ctypes.c_uint32(x)))


def encode(m, coeffs):
    c = np.ascontiguousarray(coeffs, np.uint16)
    proof = np.zeros(2 + 2 * len(c), np.uint8)
    lib().oracle_encode(ctypes.c_uint32(m), _ptr(c), len(c), _ptr(proof))
    return proof


def decode(proof):
    """-> (status, k, m, coeffs)."""
    proof = np.ascontiguousarray(proof, np.uint8)
    k = ctypes.c_int(0)
    m = ctypes.c_uint32(0)
    c = np.zeros(max(1, len(proof) // 2), np.uint16)
    st = lib().oracle_decode(_ptr(proof), ctypes.c_int64(len(proof)), ctypes.byref(k), ctypes.byref(m),
                             _ptr(c))
    return st, k.value, m.value, c[:k.value]


def mod_inverse32(a):
    return int(lib().oracle_mod_inverse32(ctypes.c_uint32(a)))


def interpolate32(x, y, lagrange=False):
    """Coefficients (ascending degree, uint32) of the polynomial through (x_j, y_j) over Z_q."""
    x = np.ascontiguousarray(x, np.uint32)
    y = np.ascontiguousarray(y, np.uint32)
    c = np.zeros(len(x), np.uint32)
    fn = lib().oracle_interpolate32_lagrange if lagrange else lib().oracle_interpolate32
    if fn(_ptr(x), _ptr(y), len(x), _ptr(c)) != 0:
        raise ValueError("x values are not distinct mod q")
    return c


def horner32(coeffs, x):
    c = np.ascontiguousarray(coeffs, np.uint32)
    return int(lib().oracle_horner32(_ptr(c), len(c), ctypes.c_uint32(x)))


def encode32(m, coeffs):
    c = np.ascontiguousarray(coeffs, np.uint32)
    proof = np.zeros(2 + 4 * len(c), np.uint8)
    lib().oracle_encode32(ctypes.c_uint32(m), _ptr(c), len(c), _ptr(proof))
    return proof


def decode32(proof):
    """-> (status, k, m, coeffs)."""
    proof = np.ascontiguousarray(proof, np.uint8)
    k = ctypes.c_int(0)
    m = ctypes.c_uint32(0)
    c = np.zeros(max(1, len(proof) // 4), np.uint32)
    st = lib().oracle_decode32(_ptr(proof), ctypes.c_int64(len(proof)), ctypes.byref(k), ctypes.byref(m),
                               _ptr(c))
    return st, k.value, m.value, c[:k.value]


def _batch_dtype_code(act, wide, padded=False):
    code = _dtype_code(act)
    if wide or padded:
        if code != 1:
            raise TypeError("the 32-bit field variant and the padded comparison are for fp32 activations")
        return 3 if padded else 2
    return code


def num_chunks(num_seqs, tokens_per_seq, chunk_len, seq_offsets=None):
    so = None if seq_offsets is None else np.ascontiguousarray(seq_offsets, np.int64)
    return int(lib().oracle_num_chunks(num_seqs, ctypes.c_int64(tokens_per_seq),
                                       None if so is None else _ptr(so), chunk_len))


def build_proofs(act, chunk_len, k, num_seqs, tokens_per_seq=0, seq_offsets=None, want_indices=True,
                 threads=None, wide=False):
    """act: 2-D [total_tokens, hidden] host array (uint16 bf16 patterns or float32).
    wide: the 32-bit field variant (fp32 only; proofs of 2 + 4k bytes).

    Returns (proofs uint8[n, 2+2k], status uint8[n], indices int32[n, k] or None), chunks in
    batch order."""
    assert act.ndim == 2 and act.strides[1] == act.itemsize
    hidden = act.shape[1]
    row_stride = act.strides[0] // act.itemsize
    so = None if seq_offsets is None else np.ascontiguousarray(seq_offsets, np.int64)
    n = num_chunks(num_seqs, tokens_per_seq, chunk_len, so)
    proofs = np.zeros((n, 2 + (4 if wide else 2) * k), np.uint8)
    status = np.zeros(n, np.uint8)
    indices = np.zeros((n, k), np.int32) if want_indices else None
    lib().oracle_build_proofs(
        _ptr(act), _batch_dtype_code(act, wide), hidden, chunk_len, k, num_seqs, ctypes.c_int64(tokens_per_seq),
        None if so is None else _ptr(so), ctypes.c_int64(row_stride), _ptr(proofs), _ptr(status),
        None if indices is None else _ptr(indices), threads or default_threads())
    return proofs, status, indices


def verify_proofs(act, proofs, chunk_len, k, num_seqs, tokens_per_seq=0, seq_offsets=None,
                  t_exp=38, t_mean=10.0, t_median=8.0, sign_in_exponent=True, gen_indices=None,
                  threads=None, wide=False, padded=False):
    """Returns a structured array (RESULT_DTYPE) with one entry per chunk.
    t_exp / t_mean / t_median: one number for the whole batch, or an array with one entry per
    chunk (thresholds chosen per generation, Section 6).
    padded: fp32 activations against 16-bit field proofs, the committed patterns padded with 16 zero
    bits and compared as fp32 (Section 5.6)."""
    assert act.ndim == 2 and act.strides[1] == act.itemsize
    hidden = act.shape[1]
    row_stride = act.strides[0] // act.itemsize
    so = None if seq_offsets is None else np.ascontiguousarray(seq_offsets, np.int64)
    n = num_chunks(num_seqs, tokens_per_seq, chunk_len, so)
    proofs = np.ascontiguousarray(proofs, np.uint8)
    assert proofs.shape == (n, 2 + (4 if wide else 2) * k)
    gi = None if gen_indices is None else np.ascontiguousarray(gen_indices, np.int32)
    results = np.zeros(n, RESULT_DTYPE)

    def each(value, dtype):
        if np.ndim(value) == 0:
            return value, None
        arr = np.ascontiguousarray(value, dtype)
        assert arr.shape == (n,)
        return 0, arr

    t_exp, exp_each = each(t_exp, np.int32)
    t_mean, mean_each = each(t_mean, np.float64)
    t_median, median_each = each(t_median, np.float64)
    lib().oracle_verify_proofs(
        _ptr(act), _batch_dtype_code(act, wide, padded), hidden, chunk_len, k, num_seqs, ctypes.c_int64(tokens_per_seq),
        None if so is None else _ptr(so), ctypes.c_int64(row_stride), _ptr(proofs), int(t_exp),
        ctypes.c_double(t_mean), ctypes.c_double(t_median), int(bool(sign_in_exponent)),
        None if exp_each is None else _ptr(exp_each), None if mean_each is None else _ptr(mean_each),
        None if median_each is None else _ptr(median_each), None if gi is None else _ptr(gi),
        _ptr(results), threads or default_threads())
    return results


def _pointer_array(arrays):
    """A C array of pointers to the given numpy arrays (None entries become NULL)."""
    out = (ctypes.c_void_p * len(arrays))()
    for i, a in enumerate(arrays):
        out[i] = None if a is None else a.ctypes.data
    return out


def build_proofs_ks(act, chunk_len, ks, num_seqs, tokens_per_seq=0, seq_offsets=None, threads=None):
    """build_proofs for several k over the same batch: each chunk is ranked once, for the largest
    k, and every k takes its prefix of that ranking (topk(h, k) is the first k of the sorted
    chunk).  16-bit field.  Returns {k: (proofs, status, indices)}."""
    assert act.ndim == 2 and act.strides[1] == act.itemsize
    hidden = act.shape[1]
    row_stride = act.strides[0] // act.itemsize
    so = None if seq_offsets is None else np.ascontiguousarray(seq_offsets, np.int64)
    n = num_chunks(num_seqs, tokens_per_seq, chunk_len, so)
    ks = [int(k) for k in ks]
    karr = np.asarray(ks, np.int32)
    proofs = [np.zeros((n, 2 + 2 * k), np.uint8) for k in ks]
    status = [np.zeros(n, np.uint8) for _ in ks]
    indices = [np.zeros((n, k), np.int32) for k in ks]
    rc = lib().oracle_build_proofs_ks(
        _ptr(act), _dtype_code(act), hidden, chunk_len, _ptr(karr), len(ks), num_seqs, ctypes.c_int64(tokens_per_seq),
        None if so is None else _ptr(so), ctypes.c_int64(row_stride), _pointer_array(proofs), _pointer_array(status),
        _pointer_array(indices), threads or default_threads())
    assert rc == 0
    return {k: (proofs[i], status[i], indices[i]) for i, k in enumerate(ks)}


def verify_proofs_ks(act, proofs_by_k, chunk_len, num_seqs, tokens_per_seq=0, seq_offsets=None, t_exp_by_k=None,
                     t_mean=10.0, t_median=8.0, sign_in_exponent=True, gen_indices_by_k=None, threads=None):
    """verify_proofs for several k over the same batch (proofs_by_k: {k: uint8[n, 2+2k]}), each
    chunk ranked once.  t_exp_by_k: {k: exponent threshold}.  Returns {k: results}."""
    assert act.ndim == 2 and act.strides[1] == act.itemsize
    hidden = act.shape[1]
    row_stride = act.strides[0] // act.itemsize
    so = None if seq_offsets is None else np.ascontiguousarray(seq_offsets, np.int64)
    n = num_chunks(num_seqs, tokens_per_seq, chunk_len, so)
    ks = [int(k) for k in proofs_by_k]
    karr = np.asarray(ks, np.int32)
    proofs = [np.ascontiguousarray(proofs_by_k[k], np.uint8) for k in ks]
    for k, pr in zip(ks, proofs):
        assert pr.shape == (n, 2 + 2 * k)
    texp = np.asarray([38 if t_exp_by_k is None else int(t_exp_by_k[k]) for k in ks], np.int32)
    gens = [None if gen_indices_by_k is None or gen_indices_by_k.get(k) is None
            else np.ascontiguousarray(gen_indices_by_k[k], np.int32) for k in ks]
    results = [np.zeros(n, RESULT_DTYPE) for _ in ks]
    rc = lib().oracle_verify_proofs_ks(
        _ptr(act), _dtype_code(act), hidden, chunk_len, _ptr(karr), len(ks), num_seqs, ctypes.c_int64(tokens_per_seq),
        None if so is None else _ptr(so), ctypes.c_int64(row_stride), _pointer_array(proofs), _ptr(texp),
        ctypes.c_double(t_mean), ctypes.c_double(t_median), int(bool(sign_in_exponent)), _pointer_array(gens),
        _pointer_array(results), threads or default_threads())
    assert rc == 0
    return {k: results[i] for i, k in enumerate(ks)}


def _chunk_spans(num_seqs, tokens_per_seq, chunk_len, seq_offsets):
    spans = []
    for s in range(num_seqs):
        begin = int(seq_offsets[s]) if seq_offsets is not None else s * tokens_per_seq
        end = int(seq_offsets[s + 1]) if seq_offsets is not None else begin + tokens_per_seq
        for r in range(begin, end, chunk_len):
            spans.append((r, min(chunk_len, end - r)))
    return spans


def commit_direct(act, chunk_len, k, num_seqs, tokens_per_seq=0, seq_offsets=None):
    """Direct commitments (Section 4: index and value stored as they are, 6 bytes per point).

    Returns (commits uint8[n, 6k], status uint8[n])."""
    assert act.ndim == 2 and act.strides[1] == act.itemsize
    hidden, row_stride, code = act.shape[1], act.strides[0] // act.itemsize, _dtype_code(act)
    spans = _chunk_spans(num_seqs, tokens_per_seq, chunk_len, seq_offsets)
    commits = np.zeros((len(spans), 6 * k), np.uint8)
    status = np.zeros(len(spans), np.uint8)
    for c, (row0, rows) in enumerate(spans):
        status[c] = lib().oracle_commit_direct_chunk(_ptr(act[row0:]), code, rows, hidden,
                                                     ctypes.c_int64(row_stride), k, _ptr(commits[c]))
    return commits, status


def verify_direct(act, commits, chunk_len, k, num_seqs, tokens_per_seq=0, seq_offsets=None,
                  t_exp=38, t_mean=10.0, t_median=8.0, sign_in_exponent=True):
    """Algorithm 2 against direct commitments.  Returns (results RESULT_DTYPE[n], exp_dev uint32[n, 9]):
    exp_dev counts, over the indices both sides selected, the exponent deviations 0, -1, +1, -2, +2,
    -10..-3, 3..10, 11..99 and >= 100 in absolute value (the columns of the table in Section 3).
    t_exp / t_mean / t_median: one number for the batch or one entry per chunk."""
    assert act.ndim == 2 and act.strides[1] == act.itemsize
    hidden, row_stride, code = act.shape[1], act.strides[0] // act.itemsize, _dtype_code(act)
    spans = _chunk_spans(num_seqs, tokens_per_seq, chunk_len, seq_offsets)
    commits = np.ascontiguousarray(commits, np.uint8)
    assert commits.shape == (len(spans), 6 * k)
    results = np.zeros(len(spans), RESULT_DTYPE)
    exp_dev = np.zeros((len(spans), 9), np.uint32)
    pick = lambda v, c: v if np.ndim(v) == 0 else v[c]
    for c, (row0, rows) in enumerate(spans):
        lib().oracle_verify_direct_chunk(
            _ptr(act[row0:]), code, rows, hidden, ctypes.c_int64(row_stride), k, _ptr(commits[c]),
            int(pick(t_exp, c)), ctypes.c_double(pick(t_mean, c)), ctypes.c_double(pick(t_median, c)),
            int(bool(sign_in_exponent)),
            _ptr(results[c:c + 1]), _ptr(exp_dev[c]))
    return results, exp_dev
