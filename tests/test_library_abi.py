"""The C-ABI library loads without a GPU, exports every symbol the header declares, and its
host-only queries behave.  No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

import paper_2501_16007_b200 as tl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built_library():
    from paper_2501_16007_b200.csrc import build
    build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "toploc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(toploc_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = tl.load_library()
    names = declared_functions()
    assert "toploc_build_proofs" in names and "toploc_verify_proofs" in names and len(names) >= 11
    for name in names:
        assert hasattr(lib, name), name
        assert hasattr(tl, name), "binding lacks %s" % name


def test_struct_sizes_match_the_header():
    assert ctypes.sizeof(tl.ToplocLayout) == 48
    assert ctypes.sizeof(tl.ToplocThresholds) == 24
    assert tl.RESULT_DTYPE.itemsize == 40


def layout(**kw):
    lay = tl.ToplocLayout()
    base = dict(dtype=0, hidden=4096, chunk_len=32, k=128, num_seqs=2, field=0, tokens_per_seq=100,
                row_stride=4096)
    base.update(kw)
    for key, val in base.items():
        setattr(lay, key, val)
    return lay


def test_constants_and_sizes():
    assert tl.toploc_get_constants() == (65521, 32769, 65536)
    assert tl.toploc_proof_bytes(128) == 258
    assert [tl.toploc_proof_bytes(k) for k in (32, 64, 256)] == [66, 130, 514]
    assert tl.toploc_status_string(0) == "ok" and "modulus" in tl.toploc_status_string(1)
    assert tl.toploc_error_string(-3).startswith("workspace")


def test_chunk_counting():
    assert tl.toploc_num_chunks(layout()) == 2 * 4          # ceil(100 / 32) per sequence
    assert tl.toploc_num_chunks(layout(tokens_per_seq=4096, num_seqs=256)) == 32768
    per_chunk = 128 * 4 + 128 * 2 + 1
    assert 8 * per_chunk <= tl.toploc_workspace_bytes(layout()) <= 8 * per_chunk + 3 * 256
    offs = np.array([0, 9, 9, 23], np.int64)
    lay = layout(num_seqs=3, chunk_len=4)
    lay.seq_offsets = offs.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))
    assert tl.toploc_num_chunks(lay) == 7
    assert tl.toploc_workspace_bytes(lay) >= 7 * 16 + 7 * per_chunk
    assert tl.toploc_staging_bytes(layout()) >= 100 * 4096 * 2 + 4 * 258


def test_the_32_bit_field_is_for_fp32_and_doubles_the_coefficients():
    wide = layout(dtype=1, field=tl.TOPLOC_FIELD_32)
    narrow = layout(dtype=1)
    assert tl.toploc_num_chunks(wide) == tl.toploc_num_chunks(narrow) == 8
    assert tl.toploc_layout_proof_bytes(wide) == 2 + 4 * 128 and tl.toploc_layout_proof_bytes(narrow) == 258
    assert tl.toploc_layout_proof_bytes(layout(k=0)) == 0
    grow = tl.toploc_workspace_bytes(wide) - tl.toploc_workspace_bytes(narrow)
    assert 8 * 128 * 2 <= grow <= 8 * 128 * 2 + 256                 # whole patterns instead of 16 bits
    assert tl.toploc_staging_bytes(wide) > tl.toploc_staging_bytes(narrow)
    thr = tl.default_thresholds(128, field=tl.TOPLOC_FIELD_32)
    assert (thr.t_exp, thr.t_mean, thr.t_median) == (8, 256.0, 128.0)
    assert tl.TOPLOC_FIELD_32_PRIME == 2 ** 32 - 5
    padded = layout(dtype=1, field=tl.TOPLOC_FIELD_16_PADDED)       # validating a bf16 model's proofs with fp32
    assert tl.toploc_layout_proof_bytes(padded) == 258
    assert tl.toploc_workspace_bytes(padded) == tl.toploc_workspace_bytes(narrow)
    lib = tl.load_library()
    assert lib.toploc_build_proofs(ctypes.c_void_p(16), ctypes.byref(padded), ctypes.c_void_p(16),
                                   ctypes.c_void_p(16), None, None, 0, None) == -2


def test_long_chunks_are_planned_in_segments():
    """A chunk above 2^19 elements is selected in segments of about 2^18 elements (whole rows) and
    merged: the scratch grows by the segments' selections and the merge's words; the chunk count
    does not change.  Only chunks that exist count against the size limit."""
    long_one = layout(hidden=4096, row_stride=4096, chunk_len=700, tokens_per_seq=700, num_seqs=1, k=128)
    assert tl.toploc_num_chunks(long_one) == 1
    segs = 11                                                     # ceil(700 * 4096 / 2^18)
    per_seg = 128 * (4 + 2 + 8) + 1 + 16
    assert tl.toploc_workspace_bytes(long_one) >= segs * per_seg + 128 * 6
    direct = layout(hidden=4096, row_stride=4096, chunk_len=128, tokens_per_seq=128, num_seqs=1, k=128)
    assert tl.toploc_workspace_bytes(direct) < 2 * 1024           # 2^19 elements: selected directly
    huge_len = layout(hidden=8192, row_stride=8192, chunk_len=1 << 30, tokens_per_seq=5000, num_seqs=2, k=128)
    assert tl.toploc_num_chunks(huge_len) == 2                    # 5000 x 8192 = 41 M elements each
    # the 24-bit index field of a candidate can force more than 64 segments: 1100 rows of 2^20
    # elements, at most 16 rows per segment -> 69 segments
    forced = layout(hidden=1 << 20, row_stride=1 << 20, chunk_len=1100, tokens_per_seq=1100, num_seqs=1, k=128)
    assert 69 * per_seg <= tl.toploc_workspace_bytes(forced) - 128 * 6 <= 69 * per_seg + 8 * 256
    lib = tl.load_library()
    assert lib.toploc_build_proofs_builtin_scratch(ctypes.c_void_p(16), ctypes.byref(long_one), ctypes.c_void_p(16),
                                                   ctypes.c_void_p(16), None, None) == -2


@pytest.mark.parametrize("bad", [dict(k=0), dict(k=513), dict(hidden=0), dict(chunk_len=0), dict(num_seqs=0),
                                 dict(dtype=7), dict(row_stride=100), dict(tokens_per_seq=0),
                                 dict(field=1), dict(field=2), dict(dtype=1, field=3), dict(dtype=1, field=-1),
                                 dict(hidden=1 << 20, chunk_len=2048, tokens_per_seq=4096, row_stride=1 << 20),
                                 dict(hidden=(1 << 24) + 8, row_stride=(1 << 24) + 8)])
def test_invalid_layouts_are_refused(bad):
    with pytest.raises(tl.ToplocError):
        tl.toploc_num_chunks(layout(**bad))


def test_device_entry_points_refuse_host_tensors():
    act = torch.zeros((64, 64), dtype=torch.bfloat16)
    lay, _ = tl.make_layout(act, 32, 8, 1, 64)
    with pytest.raises(tl.ToplocError):
        tl.toploc_build_proofs(act, lay)


def test_null_pointers_are_refused_before_any_cuda_call():
    lib = tl.load_library()
    lay = layout()
    assert lib.toploc_build_proofs(None, ctypes.byref(lay), None, None, None, None, 0, None) == -1
    thr = tl.default_thresholds()
    assert lib.toploc_verify_proofs(None, ctypes.byref(lay), None, ctypes.byref(thr), None, None, None, 0,
                                    None) == -1
    assert lib.toploc_build_proofs_host(None, ctypes.byref(lay), None, None, None, 0, None) == -1


def test_misaligned_pointers_are_refused_before_any_cuda_call():
    """A pointer a kernel would dereference with 2- or 4-byte loads must be a multiple of that size;
    the entry points say so with a return code instead of launching a kernel that would fault."""
    lib = tl.load_library()
    vp = ctypes.c_void_p
    ok = 1 << 20                                        # a 16-byte aligned address (never dereferenced here)
    bf16, fp32 = layout(), layout(dtype=1)
    thr = tl.default_thresholds()

    def build(act, lay, indices=None):
        return lib.toploc_build_proofs(vp(act), ctypes.byref(lay), vp(ok), vp(ok), indices, vp(ok), 1 << 30, None)

    def verify(act, lay, gen=None, results=ok):
        return lib.toploc_verify_proofs(vp(act), ctypes.byref(lay), vp(ok), ctypes.byref(thr), vp(results), gen,
                                        vp(ok), 1 << 30, None)

    assert build(ok + 1, bf16) == -1 and build(ok + 2, fp32) == -1 and build(ok + 3, fp32) == -1
    assert build(ok, bf16, vp(ok + 2)) == -1            # int32 indices at a 2-byte offset
    assert verify(ok + 1, bf16) == -1 and verify(ok + 2, fp32) == -1
    assert verify(ok, bf16, gen=vp(ok + 1)) == -1 and verify(ok, bf16, results=ok + 4) == -1
    assert lib.toploc_select_topk(vp(ok + 1), ctypes.byref(bf16), vp(ok), vp(ok), vp(ok), None, vp(ok), 1 << 30,
                                  None) == -1
    assert lib.toploc_select_topk(vp(ok), ctypes.byref(bf16), vp(ok), vp(ok), vp(ok), vp(ok + 2), vp(ok), 1 << 30,
                                  None) == -1
    assert lib.toploc_stream_append(vp(ok + 1), ctypes.byref(bf16), 0, vp(ok), None) == -1
    assert lib.toploc_stream_append(vp(ok + 2), ctypes.byref(fp32), 0, vp(ok), None) == -1
    assert lib.toploc_stream_finish(vp(ok), ctypes.byref(bf16), vp(ok), vp(ok), vp(ok + 2), vp(ok), 1 << 30,
                                    None) == -1
    assert lib.toploc_verify_proofs_per_chunk_thresholds(vp(ok), ctypes.byref(bf16), vp(ok), vp(ok + 4), vp(ok),
                                                         None, vp(ok), 1 << 30, None) == -1
    assert lib.toploc_commit_direct(vp(ok + 1), ctypes.byref(layout(hidden=1001, row_stride=1001)), vp(ok), vp(ok),
                                    None) == -1


def test_default_thresholds_come_from_the_library():
    t = tl.toploc_default_thresholds()
    assert (t.t_exp, t.sign_in_exponent, t.t_mean, t.t_median) == (38, 1, 10.0, 8.0)      # Section 5.2, k = 128
    assert [tl.toploc_default_thresholds(k).t_exp for k in (32, 64, 256, 512)] == [9, 19, 76, 152]
    w = tl.toploc_default_thresholds(128, tl.TOPLOC_FIELD_32)
    assert (w.t_exp, w.t_mean, w.t_median) == (8, 256.0, 128.0)
    assert tl.toploc_default_thresholds(64, tl.TOPLOC_FIELD_16_PADDED).t_exp == 4
    lib = tl.load_library()
    assert lib.toploc_default_thresholds(0, 0, ctypes.byref(t)) == -1
    assert lib.toploc_default_thresholds(128, 9, ctypes.byref(t)) == -1
    assert lib.toploc_default_thresholds(128, 0, None) == -1
    assert tl.THRESHOLDS_DTYPE.itemsize == ctypes.sizeof(tl.ToplocThresholds)


def test_negative_exponent_threshold_is_refused_by_both_validators():
    lib = tl.load_library()
    vp = ctypes.c_void_p
    ok = 1 << 20
    lay = layout()
    thr = tl.default_thresholds()
    thr.t_exp = -1
    assert lib.toploc_verify_proofs(vp(ok), ctypes.byref(lay), vp(ok), ctypes.byref(thr), vp(ok), None, vp(ok),
                                    1 << 30, None) == -1
    assert lib.toploc_verify_direct(vp(ok), ctypes.byref(lay), vp(ok), ctypes.byref(thr), vp(ok), None, None) == -1
    assert "host memory" in tl.toploc_error_string(-7)
