"""Python view of include/toploc.h: same names, argument marshalling only.

Every step of the proof path runs in the CUDA library (csrc/libtoploc.so).  torch is
used for device memory and streams, nothing else.  There is no fallback: if the library
is missing or the arguments are wrong, the call raises.
"""
import ctypes
import os

import numpy as np
import torch

__all__ = [
    "TOPLOC_DTYPE_BF16", "TOPLOC_DTYPE_FP32", "TOPLOC_MAX_K", "RESULT_DTYPE", "ToplocError",
    "ToplocLayout", "ToplocThresholds", "make_layout", "library_path", "load_library",
    "toploc_num_chunks", "toploc_proof_bytes", "toploc_layout_proof_bytes", "toploc_workspace_bytes",
    "toploc_staging_bytes", "toploc_stream_state_bytes", "toploc_stream_workspace_bytes", "toploc_stream_begin",
    "toploc_stream_append", "toploc_stream_finish", "TOPLOC_FIELD_16", "TOPLOC_FIELD_32", "TOPLOC_FIELD_16_PADDED", "TOPLOC_FIELD_32_PRIME",
    "toploc_get_constants", "toploc_status_string", "toploc_error_string",
    "toploc_build_proofs", "toploc_verify_proofs", "toploc_build_proofs_host",
    "toploc_verify_proofs_host", "toploc_build_proofs_builtin_scratch", "TOPLOC_BUILTIN_SCRATCH_BYTES", "toploc_select_topk",
    "TOPLOC_MAX_K_DIRECT", "toploc_direct_commit_bytes", "toploc_commit_direct", "toploc_verify_direct",
    "toploc_default_thresholds", "toploc_verify_proofs_per_chunk_thresholds",
    "toploc_verify_direct_per_chunk_thresholds", "THRESHOLDS_DTYPE", "thresholds_tensor",
    "toploc_rmsnorm_append",
]

TOPLOC_DTYPE_BF16 = 0
TOPLOC_FIELD_16 = 0
TOPLOC_FIELD_32 = 1
TOPLOC_FIELD_16_PADDED = 2   # validation only: fp32 activations against 16-bit field proofs
TOPLOC_FIELD_32_PRIME = 4294967291
TOPLOC_DTYPE_FP32 = 1
TOPLOC_MAX_K = 512
TOPLOC_MAX_K_DIRECT = 4096
TOPLOC_BUILTIN_SCRATCH_BYTES = 8 << 20

RESULT_DTYPE = np.dtype([
    ("exp_mismatch", "<u4"), ("n_match", "<u4"), ("mant_diff_sum", "<u4"), ("topk_mismatch", "<i4"),
    ("mant_mean", "<f8"), ("mant_median", "<f8"), ("modulus", "<u4"),
    ("accept", "u1"), ("status", "u1"), ("pad", "u1", (2,)),
])


# toploc_thresholds as a numpy record: the layout of one entry of a per-chunk threshold array
THRESHOLDS_DTYPE = np.dtype([("t_exp", "<i4"), ("sign_in_exponent", "<i4"), ("t_mean", "<f8"), ("t_median", "<f8")])


class ToplocError(RuntimeError):
    pass


class ToplocLayout(ctypes.Structure):
    _fields_ = [
        ("dtype", ctypes.c_int32), ("hidden", ctypes.c_int32), ("chunk_len", ctypes.c_int32),
        ("k", ctypes.c_int32), ("num_seqs", ctypes.c_int32), ("field", ctypes.c_int32),
        ("tokens_per_seq", ctypes.c_int64), ("seq_offsets", ctypes.POINTER(ctypes.c_int64)),
        ("row_stride", ctypes.c_int64),
    ]


class ToplocThresholds(ctypes.Structure):
    _fields_ = [
        ("t_exp", ctypes.c_int32), ("sign_in_exponent", ctypes.c_int32),
        ("t_mean", ctypes.c_double), ("t_median", ctypes.c_double),
    ]


_LIB = None


def library_path():
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "csrc", "libtoploc.so")


def load_library():
    """Loads csrc/libtoploc.so (built by csrc/build.py); raises if it is not there."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise ToplocError(
            "%s is missing: build it with `python -m paper_2501_16007_b200.csrc.build` "
            "(there is no CPU fallback)" % path)
    lib = ctypes.CDLL(path)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    lay_p, thr_p = ctypes.POINTER(ToplocLayout), ctypes.POINTER(ToplocThresholds)
    lib.toploc_num_chunks.restype, lib.toploc_num_chunks.argtypes = i64, [lay_p]
    lib.toploc_proof_bytes.restype, lib.toploc_proof_bytes.argtypes = sz, [i32]
    lib.toploc_layout_proof_bytes.restype = sz
    lib.toploc_layout_proof_bytes.argtypes = [lay_p]
    lib.toploc_stream_state_bytes.restype, lib.toploc_stream_state_bytes.argtypes = sz, [lay_p]
    lib.toploc_stream_workspace_bytes.restype, lib.toploc_stream_workspace_bytes.argtypes = sz, [lay_p]
    lib.toploc_stream_begin.restype, lib.toploc_stream_begin.argtypes = ctypes.c_int, [vp, lay_p, vp]
    lib.toploc_stream_append.restype, lib.toploc_stream_append.argtypes = ctypes.c_int, [vp, lay_p, i32, vp, vp]
    lib.toploc_stream_finish.restype = ctypes.c_int
    lib.toploc_stream_finish.argtypes = [vp, lay_p, vp, vp, vp, vp, sz, vp]
    lib.toploc_workspace_bytes.restype, lib.toploc_workspace_bytes.argtypes = sz, [lay_p]
    lib.toploc_staging_bytes.restype, lib.toploc_staging_bytes.argtypes = sz, [lay_p]
    lib.toploc_get_constants.restype = None
    lib.toploc_get_constants.argtypes = [ctypes.POINTER(ctypes.c_uint32)] * 3
    lib.toploc_status_string.restype, lib.toploc_status_string.argtypes = ctypes.c_char_p, [ctypes.c_int]
    lib.toploc_error_string.restype, lib.toploc_error_string.argtypes = ctypes.c_char_p, [ctypes.c_int]
    lib.toploc_build_proofs.restype = ctypes.c_int
    lib.toploc_build_proofs.argtypes = [vp, lay_p, vp, vp, vp, vp, sz, vp]
    lib.toploc_verify_proofs.restype = ctypes.c_int
    lib.toploc_verify_proofs.argtypes = [vp, lay_p, vp, thr_p, vp, vp, vp, sz, vp]
    lib.toploc_build_proofs_host.restype = ctypes.c_int
    lib.toploc_build_proofs_host.argtypes = [vp, lay_p, vp, vp, vp, sz, vp]
    lib.toploc_verify_proofs_host.restype = ctypes.c_int
    lib.toploc_verify_proofs_host.argtypes = [vp, lay_p, vp, thr_p, vp, vp, sz, vp]
    lib.toploc_select_topk.restype = ctypes.c_int
    lib.toploc_select_topk.argtypes = [vp, lay_p, vp, vp, vp, vp, vp, sz, vp]
    lib.toploc_build_proofs_builtin_scratch.restype = ctypes.c_int
    lib.toploc_build_proofs_builtin_scratch.argtypes = [vp, lay_p, vp, vp, vp, vp]
    lib.toploc_direct_commit_bytes.restype, lib.toploc_direct_commit_bytes.argtypes = sz, [i32]
    lib.toploc_commit_direct.restype = ctypes.c_int
    lib.toploc_commit_direct.argtypes = [vp, lay_p, vp, vp, vp]
    lib.toploc_verify_direct.restype = ctypes.c_int
    lib.toploc_verify_direct.argtypes = [vp, lay_p, vp, thr_p, vp, vp, vp]
    lib.toploc_verify_proofs_per_chunk_thresholds.restype = ctypes.c_int
    lib.toploc_verify_proofs_per_chunk_thresholds.argtypes = [vp, lay_p, vp, vp, vp, vp, vp, sz, vp]
    lib.toploc_verify_direct_per_chunk_thresholds.restype = ctypes.c_int
    lib.toploc_verify_direct_per_chunk_thresholds.argtypes = [vp, lay_p, vp, vp, vp, vp, vp]
    lib.toploc_rmsnorm_append.restype = ctypes.c_int
    lib.toploc_rmsnorm_append.argtypes = [vp, i64, vp, ctypes.c_float, lay_p, i32, vp, vp, vp]
    lib.toploc_default_thresholds.restype = ctypes.c_int
    lib.toploc_default_thresholds.argtypes = [i32, i32, thr_p]
    _LIB = lib
    return lib


def _check(rc, what):
    if rc != 0:
        raise ToplocError("%s failed: %s (%d)" % (what, toploc_error_string(rc), rc))


def _dtype_code(t):
    if t.dtype == torch.bfloat16:
        return TOPLOC_DTYPE_BF16
    if t.dtype == torch.float32:
        return TOPLOC_DTYPE_FP32
    raise ToplocError("activations must be bfloat16 or float32, got %s" % t.dtype)


def make_layout(act, chunk_len, k, num_seqs, tokens_per_seq=0, seq_offsets=None, field=TOPLOC_FIELD_16):
    """Layout of a 2-D activation tensor [total_tokens, hidden] (last dimension contiguous).
    field=TOPLOC_FIELD_32 (float32 activations only): whole patterns over Z_q, proofs of 2 + 4k bytes.

    Returns (layout, keepalive): keepalive holds the host seq_offsets array the struct points to."""
    if act.dim() != 2 or act.stride(1) != 1:
        raise ToplocError("activations must be 2-D with a contiguous last dimension")
    lay = ToplocLayout()
    lay.dtype = _dtype_code(act)
    lay.hidden = act.shape[1]
    lay.chunk_len = chunk_len
    lay.k = k
    lay.num_seqs = num_seqs
    lay.field = field
    lay.tokens_per_seq = tokens_per_seq
    lay.row_stride = act.stride(0) if act.shape[0] > 1 else act.shape[1]
    keep = None
    if seq_offsets is not None:
        keep = np.ascontiguousarray(seq_offsets, np.int64)
        if keep.shape != (num_seqs + 1,):
            raise ToplocError("seq_offsets must have num_seqs + 1 entries")
        lay.seq_offsets = keep.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))
        total = int(keep[-1])
    else:
        total = num_seqs * tokens_per_seq
    if total > act.shape[0]:
        raise ToplocError("layout describes %d rows, tensor has %d" % (total, act.shape[0]))
    return lay, keep


def toploc_num_chunks(lay):
    n = load_library().toploc_num_chunks(ctypes.byref(lay))
    if n < 0:
        raise ToplocError("invalid layout: %s" % toploc_error_string(int(n)))
    return int(n)


def toploc_proof_bytes(k):
    return int(load_library().toploc_proof_bytes(k))


def toploc_layout_proof_bytes(lay):
    return int(load_library().toploc_layout_proof_bytes(ctypes.byref(lay)))


def toploc_workspace_bytes(lay):
    return int(load_library().toploc_workspace_bytes(ctypes.byref(lay)))


def toploc_staging_bytes(lay):
    return int(load_library().toploc_staging_bytes(ctypes.byref(lay)))


def toploc_get_constants():
    p, lo, hi = ctypes.c_uint32(), ctypes.c_uint32(), ctypes.c_uint32()
    load_library().toploc_get_constants(ctypes.byref(p), ctypes.byref(lo), ctypes.byref(hi))
    return p.value, lo.value, hi.value


def toploc_status_string(code):
    return load_library().toploc_status_string(int(code)).decode()


def toploc_error_string(code):
    return load_library().toploc_error_string(int(code)).decode()


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dev_ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _workspace(lay, workspace, device):
    need = toploc_workspace_bytes(lay)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=device)
    return workspace, (0 if workspace is None else workspace.numel() * workspace.element_size())


def toploc_build_proofs(act, lay, proofs=None, status=None, indices=None, workspace=None, stream=None,
                        want_indices=False):
    """Enqueues proof generation for the batch `lay` describes on `stream` (default: torch's
    current stream).  act: CUDA tensor.  Output tensors are allocated when not given.
    Returns (proofs uint8[n, 2+2k], status uint8[n], indices int32[n, k] or None)."""
    if not act.is_cuda:
        raise ToplocError("toploc_build_proofs needs a CUDA tensor (use toploc_build_proofs_host)")
    n = toploc_num_chunks(lay)
    pb = toploc_layout_proof_bytes(lay)
    dev = act.device
    if proofs is None:
        proofs = torch.empty((n, pb), dtype=torch.uint8, device=dev)
    if status is None:
        status = torch.empty((n,), dtype=torch.uint8, device=dev)
    if indices is None and want_indices:
        indices = torch.empty((n, lay.k), dtype=torch.int32, device=dev)
    assert proofs.is_contiguous() and proofs.numel() == n * pb and status.numel() == n
    assert indices is None or (indices.is_contiguous() and indices.numel() == n * lay.k
                               and indices.dtype == torch.int32)
    workspace, wbytes = _workspace(lay, workspace, dev)
    with torch.cuda.device(dev):
        rc = load_library().toploc_build_proofs(
            _dev_ptr(act), ctypes.byref(lay), _dev_ptr(proofs), _dev_ptr(status), _dev_ptr(indices),
            _dev_ptr(workspace), wbytes, _stream_ptr(stream))
    _check(rc, "toploc_build_proofs")
    return proofs, status, indices


def toploc_verify_proofs(act, lay, proofs, thresholds=None, results=None, gen_indices=None,
                         workspace=None, stream=None):
    """Enqueues validation.  Returns a uint8 CUDA tensor [n, 40]; view it on the host with
    results.cpu().numpy().view(RESULT_DTYPE).reshape(-1)."""
    if not act.is_cuda:
        raise ToplocError("toploc_verify_proofs needs a CUDA tensor (use toploc_verify_proofs_host)")
    n = toploc_num_chunks(lay)
    dev = act.device
    thr = thresholds if thresholds is not None else default_thresholds()
    if results is None:
        results = torch.empty((n, RESULT_DTYPE.itemsize), dtype=torch.uint8, device=dev)
    assert proofs.is_contiguous() and proofs.numel() == n * toploc_layout_proof_bytes(lay)
    assert results.is_contiguous() and results.numel() == n * RESULT_DTYPE.itemsize
    assert gen_indices is None or (gen_indices.is_contiguous() and gen_indices.dtype == torch.int32
                                   and gen_indices.numel() == n * lay.k)
    workspace, wbytes = _workspace(lay, workspace, dev)
    with torch.cuda.device(dev):
        rc = load_library().toploc_verify_proofs(
            _dev_ptr(act), ctypes.byref(lay), _dev_ptr(proofs), ctypes.byref(thr), _dev_ptr(results),
            _dev_ptr(gen_indices), _dev_ptr(workspace), wbytes, _stream_ptr(stream))
    _check(rc, "toploc_verify_proofs")
    return results


def toploc_default_thresholds(k=128, field=TOPLOC_FIELD_16):
    """The library's default thresholds for a proof of k points (Section 5.2; see the header)."""
    thr = ToplocThresholds()
    _check(load_library().toploc_default_thresholds(int(k), int(field), ctypes.byref(thr)), "toploc_default_thresholds")
    return thr


def default_thresholds(k=128, sign_in_exponent=True, field=TOPLOC_FIELD_16):
    """toploc_default_thresholds with the sign-bit reading chosen by the caller."""
    thr = toploc_default_thresholds(k, field)
    thr.sign_in_exponent = 1 if sign_in_exponent else 0
    return thr


__all__.append("default_thresholds")


def thresholds_tensor(t_exp, t_mean, t_median, sign_in_exponent, device):
    """Packs per-chunk thresholds (equal-length sequences) into a CUDA uint8 tensor laid out as
    toploc_thresholds[n], for the *_per_chunk_thresholds entry points."""
    n = len(t_exp)
    rec = np.zeros(n, THRESHOLDS_DTYPE)
    rec["t_exp"], rec["t_mean"], rec["t_median"] = t_exp, t_mean, t_median
    rec["sign_in_exponent"] = sign_in_exponent
    return torch.from_numpy(rec.view(np.uint8).reshape(n, THRESHOLDS_DTYPE.itemsize)).to(device)


def toploc_verify_proofs_per_chunk_thresholds(act, lay, proofs, thresholds, results=None, gen_indices=None,
                                              workspace=None, stream=None):
    """toploc_verify_proofs with one toploc_thresholds entry per chunk: `thresholds` is a CUDA uint8
    tensor [n, 24] (see thresholds_tensor).  Returns the results tensor [n, 40]."""
    if not act.is_cuda or not thresholds.is_cuda:
        raise ToplocError("toploc_verify_proofs_per_chunk_thresholds needs CUDA tensors")
    n = toploc_num_chunks(lay)
    dev = act.device
    if results is None:
        results = torch.empty((n, RESULT_DTYPE.itemsize), dtype=torch.uint8, device=dev)
    assert proofs.is_contiguous() and proofs.numel() == n * toploc_layout_proof_bytes(lay)
    assert thresholds.is_contiguous() and thresholds.numel() * thresholds.element_size() == n * THRESHOLDS_DTYPE.itemsize
    assert results.is_contiguous() and results.numel() == n * RESULT_DTYPE.itemsize
    workspace, wbytes = _workspace(lay, workspace, dev)
    with torch.cuda.device(dev):
        rc = load_library().toploc_verify_proofs_per_chunk_thresholds(
            _dev_ptr(act), ctypes.byref(lay), _dev_ptr(proofs), _dev_ptr(thresholds), _dev_ptr(results),
            _dev_ptr(gen_indices), _dev_ptr(workspace), wbytes, _stream_ptr(stream))
    _check(rc, "toploc_verify_proofs_per_chunk_thresholds")
    return results


def toploc_build_proofs_host(act, lay, proofs, status, staging, stream=None):
    """Host-memory variant: act / proofs / status are CPU tensors (pinned for asynchronous
    copies), staging is a CUDA uint8 tensor of at least toploc_staging_bytes(lay) bytes.
    Blocks until the host outputs are complete."""
    if act.is_cuda or proofs.is_cuda or status.is_cuda or not staging.is_cuda:
        raise ToplocError("host variant: act/proofs/status on the CPU, staging on the GPU")
    with torch.cuda.device(staging.device):
        rc = load_library().toploc_build_proofs_host(
            _dev_ptr(act), ctypes.byref(lay), _dev_ptr(proofs), _dev_ptr(status), _dev_ptr(staging),
            staging.numel() * staging.element_size(), _stream_ptr(stream))
    _check(rc, "toploc_build_proofs_host")
    return proofs, status


def toploc_verify_proofs_host(act, lay, proofs, thresholds, results, staging, stream=None):
    if act.is_cuda or proofs.is_cuda or results.is_cuda or not staging.is_cuda:
        raise ToplocError("host variant: act/proofs/results on the CPU, staging on the GPU")
    thr = thresholds if thresholds is not None else default_thresholds(lay.k)
    with torch.cuda.device(staging.device):
        rc = load_library().toploc_verify_proofs_host(
            _dev_ptr(act), ctypes.byref(lay), _dev_ptr(proofs), ctypes.byref(thr), _dev_ptr(results),
            _dev_ptr(staging), staging.numel() * staging.element_size(), _stream_ptr(stream))
    _check(rc, "toploc_verify_proofs_host")
    return results


def toploc_build_proofs_builtin_scratch(act, lay, proofs, status, indices=None, stream=None):
    """Proof generation without a workspace argument: the scratch is a fixed buffer inside the
    library (TOPLOC_BUILTIN_SCRATCH_BYTES), for embedders that cannot allocate device memory
    where proofs are made.  This wrapper allocates nothing either: every output tensor must be
    passed in.  Batches whose scratch need exceeds the buffer, and ragged batches, are refused.
    Calls share the buffer: keep calls that could overlap on the GPU ordered."""
    if not act.is_cuda:
        raise ToplocError("toploc_build_proofs_builtin_scratch needs CUDA tensors")
    with torch.cuda.device(act.device):
        rc = load_library().toploc_build_proofs_builtin_scratch(
            _dev_ptr(act), ctypes.byref(lay), _dev_ptr(proofs), _dev_ptr(status), _dev_ptr(indices),
            _stream_ptr(stream))
    _check(rc, "toploc_build_proofs_builtin_scratch")
    return proofs, status, indices


def toploc_select_topk(act, lay, sel_indices=None, sel_patterns=None, status=None, ranked_indices=None,
                       workspace=None, stream=None, want_ranked=False):
    """The selection step alone.  Returns (sel_indices int32-viewable uint32 [n, k] as an int32
    tensor, sel_patterns int16 tensor holding the 16-bit patterns [n, k], status uint8 [n],
    ranked_indices int32 [n, k] or None)."""
    if not act.is_cuda:
        raise ToplocError("toploc_select_topk needs a CUDA tensor")
    n = toploc_num_chunks(lay)
    dev = act.device
    if sel_indices is None:
        sel_indices = torch.empty((n, lay.k), dtype=torch.int32, device=dev)
    if sel_patterns is None:
        sel_patterns = torch.empty((n, lay.k), dtype=torch.int16, device=dev)
    if status is None:
        status = torch.empty((n,), dtype=torch.uint8, device=dev)
    if ranked_indices is None and want_ranked:
        ranked_indices = torch.empty((n, lay.k), dtype=torch.int32, device=dev)
    workspace, wbytes = _workspace(lay, workspace, dev)
    with torch.cuda.device(dev):
        rc = load_library().toploc_select_topk(
            _dev_ptr(act), ctypes.byref(lay), _dev_ptr(sel_indices), _dev_ptr(sel_patterns), _dev_ptr(status),
            _dev_ptr(ranked_indices), _dev_ptr(workspace), wbytes, _stream_ptr(stream))
    _check(rc, "toploc_select_topk")
    return sel_indices, sel_patterns, status, ranked_indices


def toploc_stream_state_bytes(lay):
    return int(load_library().toploc_stream_state_bytes(ctypes.byref(lay)))


def toploc_stream_workspace_bytes(lay):
    return int(load_library().toploc_stream_workspace_bytes(ctypes.byref(lay)))


def toploc_stream_begin(state, lay, stream=None):
    """Empties the running selections held in `state` (a CUDA uint8 tensor of
    toploc_stream_state_bytes(lay) bytes): the start of a chunk for every sequence."""
    with torch.cuda.device(state.device):
        rc = load_library().toploc_stream_begin(_dev_ptr(state), ctypes.byref(lay), _stream_ptr(stream))
    _check(rc, "toploc_stream_begin")
    return state


def toploc_stream_append(rows, lay, token_in_chunk, state, stream=None):
    """rows: CUDA tensor [num_seqs, hidden], row `token_in_chunk` of every sequence's running chunk."""
    if not rows.is_cuda:
        raise ToplocError("toploc_stream_append needs CUDA tensors")
    with torch.cuda.device(rows.device):
        rc = load_library().toploc_stream_append(_dev_ptr(rows), ctypes.byref(lay), int(token_in_chunk),
                                                 _dev_ptr(state), _stream_ptr(stream))
    _check(rc, "toploc_stream_append")


def toploc_stream_finish(state, lay, proofs=None, status=None, indices=None, workspace=None, stream=None,
                         want_indices=False):
    """Proofs of the chunks as they stand.  Returns (proofs uint8[num_seqs, proof bytes],
    status uint8[num_seqs], indices int32[num_seqs, k] or None)."""
    dev = state.device
    n, pb = lay.num_seqs, toploc_layout_proof_bytes(lay)
    if proofs is None:
        proofs = torch.empty((n, pb), dtype=torch.uint8, device=dev)
    if status is None:
        status = torch.empty((n,), dtype=torch.uint8, device=dev)
    if indices is None and want_indices:
        indices = torch.empty((n, lay.k), dtype=torch.int32, device=dev)
    if workspace is None:
        workspace = torch.empty(max(16, toploc_stream_workspace_bytes(lay)), dtype=torch.uint8, device=dev)
    with torch.cuda.device(dev):
        rc = load_library().toploc_stream_finish(
            _dev_ptr(state), ctypes.byref(lay), _dev_ptr(proofs), _dev_ptr(status), _dev_ptr(indices),
            _dev_ptr(workspace), workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    _check(rc, "toploc_stream_finish")
    return proofs, status, indices


def toploc_direct_commit_bytes(k):
    return int(load_library().toploc_direct_commit_bytes(k))


def _direct_chunks(lay):
    # uniform batches only (the entry points refuse the others)
    return lay.num_seqs * ((lay.tokens_per_seq + lay.chunk_len - 1) // lay.chunk_len)


def toploc_commit_direct(act, lay, commits=None, status=None, stream=None):
    """Direct commitments (Section 4: index and value as they are, 6 bytes per point), k up to
    TOPLOC_MAX_K_DIRECT.  Returns (commits uint8 [n, 6k], status uint8 [n])."""
    if not act.is_cuda:
        raise ToplocError("toploc_commit_direct needs a CUDA tensor")
    n, dev = _direct_chunks(lay), act.device
    if commits is None:
        commits = torch.empty((n, 6 * lay.k), dtype=torch.uint8, device=dev)
    if status is None:
        status = torch.empty((n,), dtype=torch.uint8, device=dev)
    assert commits.is_contiguous() and commits.numel() == n * 6 * lay.k and status.numel() == n
    with torch.cuda.device(dev):
        rc = load_library().toploc_commit_direct(_dev_ptr(act), ctypes.byref(lay), _dev_ptr(commits),
                                                 _dev_ptr(status), _stream_ptr(stream))
    _check(rc, "toploc_commit_direct")
    return commits, status


def toploc_verify_direct(act, lay, commits, thresholds=None, results=None, exp_dev=None, want_exp_dev=True,
                         stream=None):
    """Validation against direct commitments.  Returns (results uint8 [n, 40] -- view with
    RESULT_DTYPE --, exp_dev int32 [n, 9] or None)."""
    if not act.is_cuda:
        raise ToplocError("toploc_verify_direct needs a CUDA tensor")
    n, dev = _direct_chunks(lay), act.device
    thr = thresholds if thresholds is not None else default_thresholds(lay.k)
    if results is None:
        results = torch.empty((n, RESULT_DTYPE.itemsize), dtype=torch.uint8, device=dev)
    if exp_dev is None and want_exp_dev:
        exp_dev = torch.empty((n, 9), dtype=torch.int32, device=dev)
    assert commits.is_contiguous() and commits.numel() == n * 6 * lay.k
    assert results.is_contiguous() and results.numel() == n * RESULT_DTYPE.itemsize
    with torch.cuda.device(dev):
        rc = load_library().toploc_verify_direct(_dev_ptr(act), ctypes.byref(lay), _dev_ptr(commits),
                                                 ctypes.byref(thr), _dev_ptr(results), _dev_ptr(exp_dev),
                                                 _stream_ptr(stream))
    _check(rc, "toploc_verify_direct")
    return results, exp_dev


def toploc_verify_direct_per_chunk_thresholds(act, lay, commits, thresholds, results=None, exp_dev=None,
                                              want_exp_dev=True, stream=None):
    """toploc_verify_direct with one toploc_thresholds entry per chunk (CUDA uint8 tensor [n, 24])."""
    if not act.is_cuda or not thresholds.is_cuda:
        raise ToplocError("toploc_verify_direct_per_chunk_thresholds needs CUDA tensors")
    n, dev = _direct_chunks(lay), act.device
    if results is None:
        results = torch.empty((n, RESULT_DTYPE.itemsize), dtype=torch.uint8, device=dev)
    if exp_dev is None and want_exp_dev:
        exp_dev = torch.empty((n, 9), dtype=torch.int32, device=dev)
    assert commits.is_contiguous() and commits.numel() == n * 6 * lay.k
    assert thresholds.is_contiguous() and thresholds.numel() * thresholds.element_size() == n * THRESHOLDS_DTYPE.itemsize
    with torch.cuda.device(dev):
        rc = load_library().toploc_verify_direct_per_chunk_thresholds(
            _dev_ptr(act), ctypes.byref(lay), _dev_ptr(commits), _dev_ptr(thresholds), _dev_ptr(results),
            _dev_ptr(exp_dev), _stream_ptr(stream))
    _check(rc, "toploc_verify_direct_per_chunk_thresholds")
    return results, exp_dev


def toploc_rmsnorm_append(x, weight, eps, lay, token_in_chunk, y, state=None, stream=None):
    """Final RMSNorm of one new row per sequence (x, y: CUDA bf16 [num_seqs, hidden]; weight: bf16
    [hidden]) that offers the normalised rows to the running selections in `state` (None: the
    normalisation alone).  See toploc_rmsnorm_append in the header."""
    if not (x.is_cuda and y.is_cuda and weight.is_cuda):
        raise ToplocError("toploc_rmsnorm_append needs CUDA tensors")
    if x.dtype != torch.bfloat16 or y.dtype != torch.bfloat16 or weight.dtype != torch.bfloat16:
        raise ToplocError("toploc_rmsnorm_append works on bfloat16 tensors")
    if x.dim() != 2 or x.stride(1) != 1 or y.stride(1) != 1 or not weight.is_contiguous():
        raise ToplocError("rows must be contiguous")
    with torch.cuda.device(x.device):
        rc = load_library().toploc_rmsnorm_append(
            _dev_ptr(x), x.stride(0) if x.shape[0] > 1 else x.shape[1], _dev_ptr(weight), float(eps),
            ctypes.byref(lay), int(token_in_chunk), _dev_ptr(y), _dev_ptr(state), _stream_ptr(stream))
    _check(rc, "toploc_rmsnorm_append")
    return y
