"""Parity of the CUDA path with the oracle for fp32 chunks committed over the 32-bit field
(TOPLOC_FIELD_32: whole patterns in Z_q, q = 2^32 - 5, proofs of 2 + 4k bytes, fp32 bit fields and the
thresholds 8 / 256 / 128 of Section 5.2 in validation)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_16007_b200 as tl
from paper_2501_16007_b200 import synth
from helpers import parity_case, gpu_build, gpu_verify, assert_build_equal, assert_results_equal, oracle_thresholds

pytestmark = pytest.mark.gpu
DEV = "cuda"
WIDE = tl.TOPLOC_FIELD_32


def noise(act, seed, rel):
    return synth.honest_noise(act, seed=seed, rel=rel)


@pytest.mark.parametrize("hidden,rows,chunk_len,k", [
    (4096, 96, 32, 128),     # the paper's shape
    (2048, 70, 32, 64),      # ragged tail: chunks of 32, 32, 6 rows
    (1000, 40, 8, 32),       # rows that are not a multiple of the tile
    (97, 64, 16, 256),       # unaligned rows (element-wise loads), largest k
    (64, 9, 4, 7),           # tiny chunks, odd k
])
def test_small_shapes(hidden, rows, chunk_len, k):
    act = synth.make_activations(2, rows, hidden, torch.float32, seed=hidden + k, device=DEV, outliers="jitter")
    # fp32 recomputation noise of a few mantissa units (accepted) and of 2^-8 (exponents hold, mantissas do not)
    rec = {"fine": noise(act, 5, 2.0 ** -22), "coarse": noise(act, 6, 2.0 ** -8)}
    _, out = parity_case(act, chunk_len, k, 2, rows, recomputed=rec, where="wide %dx%d" % (rows, hidden), wide=True)
    assert out["same"]["accept"].all() and not out["same"]["mant_diff_sum"].any()


def test_verdicts_follow_the_fp32_thresholds():
    act = synth.make_activations(4, 64, 4096, torch.float32, seed=77, device=DEV, outliers="none")
    rec = {"fine": noise(act, 8, 2.0 ** -22), "coarse": noise(act, 9, 2.0 ** -8)}
    _, out = parity_case(act, 32, 128, 4, 64, recomputed=rec, where="verdicts", wide=True)
    assert out["fine"]["accept"].all()                      # a few units of 2^-23: mean far below 256
    assert not out["coarse"]["accept"].any()                # what passes the bf16 thresholds fails these
    assert (out["coarse"]["mant_mean"] > 256.0).all()


def test_outlier_ties_and_degenerate_chunks():
    fixed = synth.make_activations(1, 64, 4096, torch.float32, seed=3, device=DEV, outliers="fixed")
    parity_case(fixed, 32, 128, 1, 64, where="wide fixed outliers", wide=True)
    equal = torch.full((64, 512), -2.5, dtype=torch.float32, device=DEV)
    parity_case(equal, 32, 128, 1, 64, where="wide equal", wide=True)
    zeros = torch.zeros((32, 256), dtype=torch.float32, device=DEV)
    parity_case(zeros, 32, 64, 1, 32, where="wide zeros", wide=True)


def test_nonfinite_patterns_short_chunks_and_malformed_proofs():
    pat = np.zeros((3, 40), np.uint32)
    pat[0, 3] = 0xFFFFFFFD      # negative NaN pattern >= q
    pat[1, 7] = 0x7FC00000      # positive NaN: ranks above everything finite
    pat[2, 1] = 0x7F800000      # +Inf
    pat[0, 10:30] = np.arange(20, dtype=np.uint32) * 0x00012345 + 0x3F800000
    act = torch.from_numpy(pat.view(np.float32)).to(DEV)
    # chunk_len 2 -> chunks of 80 and 40 elements; k = 64 exceeds the second
    g = gpu_build(act, 2, 64, 1, 3, field=WIDE)
    r = oracle.build_proofs(pat, 2, 64, 1, 3, wide=True)
    assert_build_equal(g, r, "wide nan")
    assert r[1].tolist() == [oracle.ST_NONFINITE, oracle.ST_K_EXCEEDS]
    kw = oracle_thresholds(64, wide=True)
    gv = gpu_verify(act, g[0], 2, 64, 1, 3, gen_indices=g[2], field=WIDE)
    rv = oracle.verify_proofs(pat, r[0], 2, 64, 1, 3, gen_indices=r[2], wide=True, **kw)
    assert_results_equal(gv, rv, "wide nan verify")
    bad = g[0].clone()
    bad[0, 2:6] = torch.tensor([0xFB, 0xFF, 0xFF, 0xFF], dtype=torch.uint8)      # coefficient = q
    gv = gpu_verify(act, bad, 2, 64, 1, 3, field=WIDE)
    rv = oracle.verify_proofs(pat, bad.cpu().numpy(), 2, 64, 1, 3, wide=True, **kw)
    assert_results_equal(gv, rv, "wide bad proof")
    assert rv["status"].tolist()[0] == oracle.ST_BAD_PROOF


def test_padded_rows_ragged_batch_and_sign_switch():
    base = synth.make_activations(1, 100, 2048 + 32, torch.float32, seed=12, device=DEV, outliers="jitter")
    offs = np.array([0, 33, 33, 100], np.int64)
    parity_case(base[:, :2048], 32, 128, 3, seq_offsets=offs, where="wide padded ragged", wide=True)
    act = synth.make_activations(1, 32, 1024, torch.float32, seed=13, device=DEV, outliers="none")
    flipped = -act
    g = gpu_build(act, 32, 64, 1, 32, field=WIDE)
    host, fh = synth.host_patterns(act), synth.host_patterns(flipped)
    r = oracle.build_proofs(host, 32, 64, 1, 32, wide=True)
    assert_build_equal(g, r, "wide sign")
    for sign_in_exponent in (True, False):
        thr = tl.default_thresholds(64, sign_in_exponent=sign_in_exponent, field=WIDE)
        gv = gpu_verify(flipped, g[0], 32, 64, 1, 32, thresholds=thr, field=WIDE)
        rv = oracle.verify_proofs(fh, r[0], 32, 64, 1, 32, wide=True,
                                  **oracle_thresholds(64, sign_in_exponent=sign_in_exponent, wide=True))
        assert_results_equal(gv, rv, "wide sign %s" % sign_in_exponent)
        assert bool(rv["accept"][0]) == (not sign_in_exponent)


def test_long_chunk_over_the_32_bit_field():
    act = synth.make_activations(1, 300, 4096, torch.float32, seed=14, device=DEV, outliers="none")
    rec = {"fine": noise(act, 15, 2.0 ** -22)}
    parity_case(act, 300, 128, 1, 300, recomputed=rec, where="wide long", wide=True)


def test_host_entry_points_and_refusals():
    act = synth.make_activations(3, 64, 1024, torch.float32, seed=16, device=DEV, outliers="jitter")
    lay, _ = tl.make_layout(act, 32, 128, 3, 64, field=WIDE)
    n, pb = tl.toploc_num_chunks(lay), tl.toploc_layout_proof_bytes(lay)
    assert pb == 2 + 4 * 128
    g = gpu_build(act, 32, 128, 3, 64, field=WIDE)
    h_act = act.cpu().pin_memory()
    h_proofs = torch.empty((n, pb), dtype=torch.uint8).pin_memory()
    h_status = torch.empty((n,), dtype=torch.uint8).pin_memory()
    staging = torch.empty(tl.toploc_staging_bytes(lay), dtype=torch.uint8, device=DEV)
    tl.toploc_build_proofs_host(h_act, lay, h_proofs, h_status, staging)
    assert torch.equal(h_proofs, g[0].cpu()) and torch.equal(h_status, g[1].cpu())
    h_res = torch.empty((n, 40), dtype=torch.uint8).pin_memory()
    tl.toploc_verify_proofs_host(h_act, lay, h_proofs, tl.default_thresholds(128, field=WIDE), h_res, staging)
    assert h_res.numpy().view(tl.RESULT_DTYPE).reshape(-1)["accept"].all()
    with pytest.raises(tl.ToplocError, match="unsupported"):
        tl.toploc_select_topk(act, lay)
    bf = act.to(torch.bfloat16)
    with pytest.raises(tl.ToplocError):
        tl.make_layout(bf, 32, 128, 3, 64, field=WIDE) and tl.toploc_num_chunks(tl.make_layout(bf, 32, 128, 3, 64, field=WIDE)[0])


def test_fp32_validator_of_a_bf16_model_pads_the_commitments():
    """Section 5.6: proofs generated from bf16 activations, validated against the fp32 activations they
    were rounded from, the committed patterns padded with 16 zero bits: exponents agree, the mantissas
    differ by what the rounding removed (thousands of fp32 units), so the fp32 thresholds reject."""
    PAD = tl.TOPLOC_FIELD_16_PADDED
    full = synth.make_activations(3, 64, 2048, torch.float32, seed=21, device=DEV, outliers="none")
    model = full.to(torch.bfloat16)                           # what the bf16 generator computed with
    g = gpu_build(model, 32, 128, 3, 64)
    r = oracle.build_proofs(synth.host_patterns(model), 32, 128, 3, 64)
    assert_build_equal(g, r, "bf16 generator")
    kw = oracle_thresholds(128, wide=True)
    for name, seen in (("fp32 original", full), ("bf16 values as fp32", model.to(torch.float32))):
        gv = gpu_verify(seen, g[0], 32, 128, 3, 64, gen_indices=g[2], field=PAD)
        rv = oracle.verify_proofs(synth.host_patterns(seen), r[0], 32, 128, 3, 64, gen_indices=r[2], padded=True, **kw)
        assert_results_equal(gv, rv, "padded " + name)
        if name.startswith("bf16"):
            assert rv["accept"].all() and not rv["mant_diff_sum"].any()
        else:
            assert not rv["accept"].any() and (rv["mant_mean"] > 256.0).all()
    # a long chunk and the host entry point take the same path
    long_full = synth.make_activations(1, 300, 4096, torch.float32, seed=22, device=DEV, outliers="none")
    long_model = long_full.to(torch.bfloat16)
    lg = gpu_build(long_model, 300, 128, 1, 300)
    lr = oracle.build_proofs(synth.host_patterns(long_model), 300, 128, 1, 300)
    gv = gpu_verify(long_full, lg[0], 300, 128, 1, 300, gen_indices=lg[2], field=PAD)
    rv = oracle.verify_proofs(synth.host_patterns(long_full), lr[0], 300, 128, 1, 300, gen_indices=lr[2], padded=True, **kw)
    assert_results_equal(gv, rv, "padded long chunk")
    lay, _ = tl.make_layout(full, 32, 128, 3, 64, field=PAD)
    with pytest.raises(tl.ToplocError, match="unsupported"):
        tl.toploc_build_proofs(full, lay)


def test_the_four_generation_validation_precision_pairs():
    """The pairs of the precision table in Section 5.6 on synthetic activations: an fp32 model passes both
    validators, a bf16 model only the bf16 one."""
    S, T, H, L, k = 2, 64, 4096, 32, 128
    full = synth.make_activations(S, T, H, torch.float32, seed=23, device=DEV, outliers="none")
    half = full.to(torch.bfloat16)
    recomputed_full = noise(full, 24, 2.0 ** -22)             # each validator recomputes with its own rounding noise
    recomputed_half = synth.honest_noise(half, seed=25)
    outcomes = {}
    # fp32 model, fp32 validator: whole patterns, fp32 thresholds
    _, out = parity_case(full, L, k, S, T, recomputed={"v": recomputed_full}, where="fp32-fp32", wide=True)
    outcomes["fp32-fp32"] = out["v"]["accept"].all()
    # fp32 model, bf16 validator: 16-bit commitments of the fp32 values, bf16 thresholds
    g = gpu_build(full, L, k, S, T)
    r = oracle.build_proofs(synth.host_patterns(full), L, k, S, T)
    assert_build_equal(g, r, "fp32 model, 16-bit field")
    gv = gpu_verify(recomputed_half, g[0], L, k, S, T, gen_indices=g[2])
    rv = oracle.verify_proofs(synth.host_patterns(recomputed_half), r[0], L, k, S, T, gen_indices=r[2],
                              **oracle_thresholds(k))
    assert_results_equal(gv, rv, "fp32-bf16")
    outcomes["fp32-bf16"] = rv["accept"].all()
    # bf16 model: bf16 validator, then fp32 validator with padded commitments
    g = gpu_build(half, L, k, S, T)
    r = oracle.build_proofs(synth.host_patterns(half), L, k, S, T)
    gv = gpu_verify(recomputed_half, g[0], L, k, S, T, gen_indices=g[2])
    rv = oracle.verify_proofs(synth.host_patterns(recomputed_half), r[0], L, k, S, T, gen_indices=r[2],
                              **oracle_thresholds(k))
    assert_results_equal(gv, rv, "bf16-bf16")
    outcomes["bf16-bf16"] = rv["accept"].all()
    gv = gpu_verify(recomputed_full, g[0], L, k, S, T, gen_indices=g[2], field=tl.TOPLOC_FIELD_16_PADDED)
    rv = oracle.verify_proofs(synth.host_patterns(recomputed_full), r[0], L, k, S, T, gen_indices=r[2], padded=True,
                              **oracle_thresholds(k, wide=True))
    assert_results_equal(gv, rv, "bf16-fp32")
    outcomes["bf16-fp32"] = rv["accept"].any()
    assert outcomes == {"fp32-fp32": True, "fp32-bf16": True, "bf16-bf16": True, "bf16-fp32": False}
