"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded bytes.  Proof bytes, selected indices, statuses and every integer statistic must be
identical; fp64 mean / median within 1e-9 (helpers.MEAN_TOL)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_16007_b200 as tl
from paper_2501_16007_b200 import synth

from helpers import (assert_build_equal, assert_results_equal, gpu_build, gpu_verify, oracle_thresholds,
                     parity_case)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def from_patterns(pat):
    """uint16 numpy patterns -> bf16 CUDA tensor with those exact bits."""
    return torch.from_numpy(pat.view(np.int16).copy()).view(torch.bfloat16).to(DEV)


# ------------------------------------------------------------------ small shapes, every code path

@pytest.mark.parametrize("hidden,rows,chunk_len,k", [
    (4096, 96, 32, 128),     # three chunks of the paper's shape
    (2048, 50, 16, 32),      # ragged last chunk (50 = 3 * 16 + 2)
    (8192, 64, 64, 256),     # 2 MiB-class chunk in fp32 terms, largest k
    (1000, 40, 8, 64),       # hidden not a multiple of 8: element-wise loads
    (64, 7, 7, 5),           # smaller than one tile
    (520, 33, 32, 128),      # 16-byte aligned rows, odd tile remainder
])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_small_shapes(hidden, rows, chunk_len, k, dtype):
    act = synth.make_activations(2, rows, hidden, dtype, seed=hidden + rows, device=DEV,
                                 outliers="jitter")
    noisy = synth.honest_noise(act, seed=5)
    other = synth.make_activations(2, rows, hidden, dtype, seed=999, device=DEV, outliers="jitter")
    parity_case(act, chunk_len, k, 2, rows, recomputed={"honest": noisy, "other": other},
                where="H%d L%d k%d %s" % (hidden, chunk_len, k, dtype))


@pytest.mark.parametrize("dtype,wide", [(torch.bfloat16, False), (torch.float32, False), (torch.float32, True)])
def test_k_512(dtype, wide):
    """The largest k of the polynomial proofs: Algorithm 6 still finds a modulus for 512 indices (a
    given candidate separates them with probability about exp(-k^2 / 2m) = 0.13), the kernels take
    their larger per-warp scratch and sixteen points per lane.  Proofs of 2 + 2k = 1026 bytes."""
    S, T, H, L, k = 2, 96, 4096, 32, 512
    act = synth.make_activations(S, T, H, dtype, seed=77, device=DEV, outliers="jitter")
    noisy = synth.honest_noise(act, seed=78, rel=2.0 ** (-22 if wide else -8))
    other = synth.make_activations(S, T, H, dtype, seed=79, device=DEV, outliers="jitter")
    r, v = parity_case(act, L, k, S, T, recomputed={"honest": noisy, "other": other}, where="k512 %s" % dtype,
                       wide=wide)
    assert r[0].shape == (6, 2 + (4 if wide else 2) * k) and not r[1].any()
    assert v["same"]["accept"].all() and not v["other"]["accept"].any()
    # ragged tail, padded rows and a k between the two scratch sizes' limits
    wide_rows = synth.make_activations(1, 70, 2048 + 64, dtype, seed=80, device=DEV, outliers="none")
    parity_case(wide_rows[:, :2048], 32, 300, 1, 70, where="k300 strided %s" % dtype, wide=wide)


def test_no_injective_modulus_is_a_status_not_a_proof():
    """Algorithm 6 ends without a modulus when the differences of the selected indices cover its
    whole search range: 512 indices (0..255 and the multiples of 256 up to 65536) do.  The chunk
    gets its status and a zero proof on both sides; its neighbour in the batch is unaffected; the
    zero proofs validate the same way on both sides."""
    idx = list(range(256)) + [256 * j for j in range(1, 257)]
    pat = np.full((64, 4096), 0x3C00, np.uint16)
    pat[:32].reshape(-1)[idx] = 0x4500                               # first chunk: no modulus exists
    rng = np.random.default_rng(3)
    pat[32:] = rng.integers(0x3000, 0x4400, size=(32, 4096)).astype(np.uint16)   # second chunk: ordinary
    act = from_patterns(pat)
    r, v = parity_case(act, 32, 512, 1, 64, where="no modulus")
    assert r[1].tolist() == [oracle.ST_NO_MODULUS, oracle.ST_OK] and not r[0][0].any() and r[0][1].any()


@pytest.mark.parametrize("outliers", ["fixed", "none"])
def test_outlier_recipes(outliers):
    act = synth.make_activations(3, 64, 4096, torch.bfloat16, seed=3, device=DEV, outliers=outliers)
    fp8 = synth.fp8_roundtrip(act)
    parity_case(act, 32, 128, 3, 64, recomputed={"fp8": fp8}, where=outliers)


def test_padded_rows_take_the_strided_path():
    wide = synth.make_activations(1, 70, 1024 + 64, torch.bfloat16, seed=8, device=DEV, outliers="none")
    act = wide[:, :1024]                       # row stride 1088, hidden 1024: aligned rows with padding
    assert not act.is_contiguous()
    parity_case(act, 32, 64, 1, 70, where="strided")
    odd = wide[:, 1:1001]                      # misaligned start: element-wise path
    host = synth.host_patterns(wide)[:, 1:1001]
    g = gpu_build(odd, 32, 64, 1, 70)
    r = oracle.build_proofs(host, 32, 64, 1, 70)
    assert_build_equal(g, r, "misaligned")


def test_ragged_batch_with_empty_sequence():
    act = synth.make_activations(1, 23 + 40, 512, torch.bfloat16, seed=12, device=DEV, outliers="jitter")
    offsets = [0, 9, 9, 23, 63]
    parity_case(act, 4, 16, 4, seq_offsets=offsets, where="ragged")


# ------------------------------------------------------------------ degenerate inputs

def test_all_equal_and_all_zero_chunks():
    for pattern in (0x0000, 0x42A0, 0x8000):
        pat = np.full((64, 2048), pattern, np.uint16)
        act = from_patterns(pat)
        g = gpu_build(act, 32, 128, 1, 64)
        r = oracle.build_proofs(pat, 32, 128, 1, 64)
        assert_build_equal(g, r, "constant %04x" % pattern)
        assert g[2].cpu().numpy()[0].tolist() == list(range(128))


def test_growing_magnitudes_overflow_the_candidate_buffer():
    # every element beats all earlier ones: the filter never rejects anything
    n = 32 * 1024
    pat = (np.arange(n, dtype=np.uint32) // 2 + 0x0100).astype(np.uint16).reshape(32, 1024)
    act = from_patterns(pat)
    g = gpu_build(act, 32, 128, 1, 32)
    r = oracle.build_proofs(pat, 32, 128, 1, 32)
    assert_build_equal(g, r, "ascending")
    # and the mirror image: the first tile already holds the answer
    pat2 = pat.reshape(-1)[::-1].copy().reshape(32, 1024)
    g = gpu_build(from_patterns(pat2), 32, 128, 1, 32)
    r = oracle.build_proofs(pat2, 32, 128, 1, 32)
    assert_build_equal(g, r, "descending")


def test_heavy_ties_at_the_cut():
    rng = np.random.default_rng(4)
    vals = rng.integers(0, 5, size=(32, 4096)).astype(np.uint16) * 0x0080 + 0x3F80  # 5 magnitudes
    vals ^= (rng.integers(0, 2, size=vals.shape).astype(np.uint16) << 15)
    act = from_patterns(vals)
    for k in (1, 7, 128, 256):
        g = gpu_build(act, 32, k, 1, 32)
        r = oracle.build_proofs(vals, 32, k, 1, 32)
        assert_build_equal(g, r, "ties k=%d" % k)


def test_subnormal_and_nonfinite_thresholds():
    """The streaming filter switches between a floating-point and an integer compare depending
    on the threshold: exercise thresholds in the subnormal range and above infinity."""
    rng = np.random.default_rng(17)
    tiny = rng.integers(0, 0x0080, size=(64, 4096)).astype(np.uint16)          # zeros and subnormals only
    tiny ^= (rng.integers(0, 2, size=tiny.shape).astype(np.uint16) << 15)
    mixed = tiny.copy()
    mixed[:, ::7] = rng.integers(0x0080, 0x0200, size=mixed[:, ::7].shape).astype(np.uint16)  # small normals
    wild = rng.integers(0x3000, 0x4400, size=(64, 4096)).astype(np.uint16)
    spots = rng.random(wild.shape) < 0.002                                      # ~500 NaN/Inf per chunk
    wild[spots] = rng.integers(0x7F80, 0x8000, size=int(spots.sum())).astype(np.uint16)
    wild ^= (rng.integers(0, 2, size=wild.shape).astype(np.uint16) << 15)
    for name, pat in (("subnormal", tiny), ("mixed", mixed), ("nonfinite", wild)):
        act = from_patterns(pat)
        for k in (128, 256):
            g = gpu_build(act, 32, k, 1, 64)
            r = oracle.build_proofs(pat, 32, k, 1, 64)
            assert_build_equal(g, r, "%s k=%d" % (name, k))


def test_chunk_smaller_than_k_and_nan_patterns():
    pat = np.zeros((3, 40), np.uint16)
    pat[0, 3] = 0xFFF5          # negative NaN pattern >= p
    pat[1, 7] = 0x7FC0          # positive NaN: ranks above everything finite
    pat[2, 1] = 0x7F80          # +Inf
    act = from_patterns(pat)
    # chunk_len 2 -> chunks of 80 and 40 elements; k = 64 exceeds the second
    g = gpu_build(act, 2, 64, 1, 3)
    r = oracle.build_proofs(pat, 2, 64, 1, 3)
    assert_build_equal(g, r, "nan")
    assert r[1].tolist() == [oracle.ST_NONFINITE, oracle.ST_K_EXCEEDS]
    gv = gpu_verify(act, g[0], 2, 64, 1, 3, gen_indices=g[2])
    rv = oracle.verify_proofs(pat, r[0], 2, 64, 1, 3, gen_indices=r[2], **oracle_thresholds(64))
    assert_results_equal(gv, rv, "nan verify")


def test_malformed_proofs_are_reported_not_trusted():
    act = synth.make_activations(1, 64, 1024, torch.bfloat16, seed=2, device=DEV)
    g = gpu_build(act, 32, 32, 1, 64)
    proofs = g[0].clone()
    proofs[0, 0], proofs[0, 1] = 0x00, 0x80      # m = 32768
    proofs[1, 4], proofs[1, 5] = 0xF1, 0xFF      # coefficient = p
    gv = gpu_verify(act, proofs, 32, 32, 1, 64)
    rv = oracle.verify_proofs(synth.host_patterns(act), proofs.cpu().numpy(), 32, 32, 1, 64,
                              **oracle_thresholds(32))
    assert_results_equal(gv, rv, "bad proof")
    assert gv["status"].tolist() == [3, 3]


def test_selection_entry_point_matches_the_oracle_topk():
    act = synth.make_activations(2, 96, 4096, torch.bfloat16, seed=41, device=DEV, outliers="jitter")
    lay, _ = tl.make_layout(act, 32, 128, 2, 96)
    idx, pat, status, ranked = tl.toploc_select_topk(act, lay, want_ranked=True)
    torch.cuda.synchronize()
    host = synth.host_patterns(act)
    idx, pat, ranked = idx.cpu().numpy(), pat.cpu().numpy().view(np.uint16), ranked.cpu().numpy()
    assert not status.any().item()
    for c in range(6):
        want_idx, want_bits = oracle.topk(host[c * 32:(c + 1) * 32], 128)
        assert ranked[c].tolist() == want_idx.tolist()
        order = np.argsort(idx[c])
        ref = np.argsort(want_idx)
        assert idx[c][order].tolist() == want_idx[ref].tolist()           # same set ...
        assert pat[c][order].tolist() == want_bits[ref].tolist()          # ... with the same values


def test_sign_bit_reading_switch():
    act = synth.make_activations(1, 64, 4096, torch.bfloat16, seed=6, device=DEV)
    other = synth.make_activations(1, 64, 4096, torch.bfloat16, seed=1006, device=DEV)
    g = gpu_build(act, 32, 128, 1, 64)
    for sign in (True, False):
        thr = tl.default_thresholds(128, sign_in_exponent=sign)
        gv = gpu_verify(other, g[0], 32, 128, 1, 64, thresholds=thr)
        rv = oracle.verify_proofs(synth.host_patterns(other), g[0].cpu().numpy(), 32, 128, 1, 64,
                                  **oracle_thresholds(128, sign))
        assert_results_equal(gv, rv, "sign=%s" % sign)


def test_host_buffer_entry_points_match_device_ones():
    act = synth.make_activations(5, 96, 2048, torch.bfloat16, seed=21, device=DEV, outliers="jitter")
    lay, _ = tl.make_layout(act, 32, 128, 5, 96)
    n = tl.toploc_num_chunks(lay)
    g = gpu_build(act, 32, 128, 5, 96)
    h_act = act.cpu().pin_memory()
    h_proofs = torch.empty((n, 258), dtype=torch.uint8).pin_memory()
    h_status = torch.empty((n,), dtype=torch.uint8).pin_memory()
    # staging for two sequences at a time: the batch goes through in three groups
    staging = torch.empty(2 * tl.toploc_staging_bytes(lay) + 4096, dtype=torch.uint8, device=DEV)
    tl.toploc_build_proofs_host(h_act, lay, h_proofs, h_status, staging)
    assert torch.equal(h_proofs, g[0].cpu()) and torch.equal(h_status, g[1].cpu())
    h_res = torch.empty((n, 40), dtype=torch.uint8).pin_memory()
    tl.toploc_verify_proofs_host(h_act, lay, h_proofs, tl.default_thresholds(), h_res, staging)
    gv = gpu_verify(act, g[0], 32, 128, 5, 96)
    hv = h_res.numpy().view(tl.RESULT_DTYPE).reshape(-1)
    assert_results_equal(hv, gv, "host variant")
    small = torch.empty(1024, dtype=torch.uint8, device=DEV)
    with pytest.raises(tl.ToplocError):
        tl.toploc_build_proofs_host(h_act, lay, h_proofs, h_status, small)


def test_host_detected_errors_leave_nothing_enqueued():
    """Bad arguments come back as error codes before any launch: a workspace that is too small or
    misaligned, an odd proof pointer, a negative threshold."""
    import ctypes
    act = synth.make_activations(1, 64, 1024, torch.bfloat16, seed=2, device=DEV)
    lay, _ = tl.make_layout(act, 32, 32, 1, 64)
    n = tl.toploc_num_chunks(lay)
    need = tl.toploc_workspace_bytes(lay)
    proofs = torch.zeros((n, 66), dtype=torch.uint8, device=DEV)
    status = torch.full((n,), 77, dtype=torch.uint8, device=DEV)
    small = torch.empty(need - 1, dtype=torch.uint8, device=DEV)
    with pytest.raises(tl.ToplocError, match="workspace"):
        tl.toploc_build_proofs(act, lay, proofs, status, workspace=small)
    big = torch.empty(need + 64, dtype=torch.uint8, device=DEV)
    with pytest.raises(tl.ToplocError, match="invalid argument"):
        tl.toploc_build_proofs(act, lay, proofs, status, workspace=big[8:])          # not 16-byte aligned
    lib = tl.load_library()
    odd = ctypes.c_void_p(proofs.data_ptr() + 1)
    rc = lib.toploc_build_proofs(ctypes.c_void_p(act.data_ptr()), ctypes.byref(lay), odd,
                                 ctypes.c_void_p(status.data_ptr()), None, ctypes.c_void_p(big.data_ptr()),
                                 need, None)
    assert rc == -1
    thr = tl.default_thresholds(32)
    thr.t_exp = -1
    with pytest.raises(tl.ToplocError, match="invalid argument"):
        tl.toploc_verify_proofs(act, lay, proofs, thr)
    torch.cuda.synchronize()
    assert (status == 77).all().item() and not proofs.any().item()                   # nothing ran


# ------------------------------------------------------------------ the named configurations

def test_config_tiny():
    """1 sequence, 4 chunks of 32 x 4096 bf16, seed 0, k = 128: generate, validate an identical
    copy and a +1-ulp copy."""
    act = synth.make_activations(1, 128, 4096, torch.bfloat16, seed=0, device=DEV)
    ulp = synth.plus_one_ulp(act, seed=0)
    r, v = parity_case(act, 32, 128, 1, 128, recomputed={"ulp": ulp}, where="tiny")
    assert r[0].shape == (4, 258)
    assert v["same"]["accept"].tolist() == [1] * 4 and not v["same"]["mant_diff_sum"].any()
    assert v["ulp"]["accept"].tolist() == [1] * 4


def test_config_8b_decode_and_validation_sweep():
    """64 sequences x 2048 tokens, H = 4096 (4096 proofs), then the validation sweep: honest
    reorder noise, other seed, fp8 round trip, 16-token prefix shift -- every chunk compared."""
    S, T, H = 64, 2048, 4096
    act = synth.make_activations(S, T, H, torch.bfloat16, seed=2, device=DEV)
    other = synth.make_activations(S, T, H, torch.bfloat16, seed=1002, device=DEV)
    rec = {
        "honest": synth.honest_noise(act, seed=3),
        "other_seed": other,
        "fp8": synth.fp8_roundtrip(act),
        "prefix_shift": synth.prefix_shift(act, other, S, T, 16),
    }
    r, v = parity_case(act, 32, 128, S, T, recomputed=rec, where="8B")
    assert r[0].shape == (4096, 258) and not r[1].any()
    assert v["same"]["accept"].all() and v["honest"]["accept"].all()
    assert not v["other_seed"]["accept"].any() and not v["prefix_shift"]["accept"].any()


def full_size_70b_case(recipe, seed, sequences):
    """Generates and validates the 70B-shaped batch (256 sequences x 4096 tokens, H = 8192, ~17 GB) in
    one call each -- the launch configuration the benchmark times -- and compares the sequences
    listed with the oracle chunk by chunk: proof bytes, statuses and indices of the build, every
    statistic and verdict of the validation against an honest-noise copy.  The oracle receives
    one sequence (64 MiB) at a time."""
    S, T, H, L, k = 256, 4096, 8192, 32, 128
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * 2 ** 30:
        pytest.skip("needs 40 GB of free device memory")
    act = synth.make_activations(S, T, H, torch.bfloat16, seed=seed, device=DEV, outliers=recipe)
    g = gpu_build(act, L, k, S, T)
    assert not g[1].any().item()
    same = gpu_verify(act, g[0], L, k, S, T, gen_indices=g[2])
    assert same["accept"].all() and not same["exp_mismatch"].any() and not same["mant_diff_sum"].any()
    assert (same["n_match"] == k).all() and not same["topk_mismatch"].any()
    assert ((same["modulus"] >= 32769) & (same["modulus"] <= 65536)).all()
    noisy = synth.honest_noise(act, seed=seed + 1)
    honest = gpu_verify(noisy, g[0], L, k, S, T, gen_indices=g[2])
    cps = T // L
    for s in sequences:
        rows = slice(s * T, (s + 1) * T)
        r = oracle.build_proofs(synth.host_patterns(act[rows]), L, k, 1, T)
        sub = tuple(t[s * cps:(s + 1) * cps] for t in g)
        assert_build_equal(sub, r, "70B %s seq %d" % (recipe, s))
        rv = oracle.verify_proofs(synth.host_patterns(noisy[rows]), r[0], L, k, 1, T, gen_indices=r[2],
                                  **oracle_thresholds(k))
        assert_results_equal(honest[s * cps:(s + 1) * cps], rv, "70B %s honest seq %d" % (recipe, s))
    return g, honest


def test_config_70b_full_size_every_chunk():
    """The literal recipe (+-80 on eight fixed channels): all 32768 chunks against the oracle."""
    full_size_70b_case("fixed", 4, range(256))


@pytest.mark.parametrize("recipe", ["jitter", "none", "rising"])
def test_config_70b_full_size_varied_selections(recipe):
    """With +-80 outliers every chunk selects the same index set (the first 128 outliers); jittered
    outlier magnitudes, plain heavy-tailed data and magnitudes that grow through every chunk make
    the selected set, the modulus and the statistics differ from chunk to chunk.  Same full-size
    launches; sixteen whole sequences (2048 chunks) against the oracle."""
    g, honest = full_size_70b_case(recipe, {"jitter": 40, "none": 41, "rising": 42}[recipe], range(7, 256, 16))
    distinct = {tuple(row) for row in g[2][:4096:64].cpu().numpy().tolist()}
    assert len(distinct) > 32, "the selected index sets should vary from chunk to chunk"


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("hidden", [2048, 4096, 8192])
def test_config_sweep(hidden, dtype):
    """k in {32, 64, 128, 256} x chunk length in {16, 32, 64} at 128 sequences x 1024 tokens.
    Every chunk of every point is compared with the oracle: proof bytes, statuses and indices of
    the build, every statistic and verdict of the validation against an honest-noise copy.  The
    oracle ranks a chunk once per chunk length and gives each k its prefix of that ranking."""
    S, T = 128, 1024
    ks = (32, 64, 128, 256)
    act = synth.make_activations(S, T, hidden, dtype, seed=50 + hidden // 1024, device=DEV)
    noisy = synth.honest_noise(act, seed=9)
    host, host_noisy = synth.host_patterns(act), synth.host_patterns(noisy)
    for chunk_len in (16, 32, 64):
        built = oracle.build_proofs_ks(host, chunk_len, ks, S, T)
        judged = oracle.verify_proofs_ks(host_noisy, {k: built[k][0] for k in ks}, chunk_len, S, T,
                                         t_exp_by_k={k: oracle_thresholds(k)["t_exp"] for k in ks},
                                         gen_indices_by_k={k: built[k][2] for k in ks})
        for k in ks:
            where = "sweep H%d L%d k%d %s" % (hidden, chunk_len, k, dtype)
            g = gpu_build(act, chunk_len, k, S, T)
            assert_build_equal(g, built[k], where)
            gv = gpu_verify(noisy, g[0], chunk_len, k, S, T, gen_indices=g[2])
            assert_results_equal(gv, judged[k], where)


def test_thresholds_per_chunk_decide_each_chunk_by_its_own_entry():
    """Section 6: thresholds chosen per generation.  One call, a thresholds entry per chunk; the
    statistics equal those of the single-threshold call, the verdicts follow each chunk's entry,
    and both agree with the oracle given the same per-chunk thresholds."""
    S, T, H, L, k = 4, 128, 2048, 32, 64
    act = synth.make_activations(S, T, H, torch.bfloat16, seed=61, device=DEV, outliers="none")
    noisy = synth.honest_noise(act, seed=62, rel=2.0 ** -6)          # coarse noise: statistics well above zero
    lay, _ = tl.make_layout(act, L, k, S, T)
    n = tl.toploc_num_chunks(lay)
    g = gpu_build(act, L, k, S, T)
    plain = gpu_verify(noisy, g[0], L, k, S, T, gen_indices=g[2])
    assert plain["exp_mismatch"].max() > 0 and plain["mant_mean"].max() > 0
    # chunk c is judged by: exponent threshold = its own mismatch count minus (c % 2), generous otherwise
    t_exp = (plain["exp_mismatch"].astype(np.int64) - (np.arange(n) % 2)).astype(np.int32)
    t_mean = np.where(np.arange(n) % 3 == 0, plain["mant_mean"] * 0.5, 1e9)
    t_median = np.full(n, 1e9)
    thr = tl.thresholds_tensor(t_exp, t_mean, t_median, 1, DEV)
    res = tl.toploc_verify_proofs_per_chunk_thresholds(noisy, lay, g[0], thr, gen_indices=g[2])
    torch.cuda.synchronize()
    got = res.cpu().numpy().view(tl.RESULT_DTYPE).reshape(-1)
    ref = oracle.verify_proofs(synth.host_patterns(noisy), g[0].cpu().numpy(), L, k, S, T, gen_indices=g[2].cpu().numpy(),
                               t_exp=t_exp, t_mean=t_mean, t_median=t_median)
    assert_results_equal(got, ref, "per-chunk thresholds")
    for f in ("exp_mismatch", "n_match", "mant_diff_sum", "topk_mismatch"):
        assert np.array_equal(got[f], plain[f])
    assert 0 < got["accept"].sum() < n                                 # both verdicts occur in the one call
    # the direct form takes the same array
    commits, _ = tl.toploc_commit_direct(act, lay)
    dres, _ = tl.toploc_verify_direct_per_chunk_thresholds(noisy, lay, commits, thr)
    torch.cuda.synchronize()
    dgot = dres.cpu().numpy().view(tl.RESULT_DTYPE).reshape(-1)
    dref, _ = oracle.verify_direct(synth.host_patterns(noisy), commits.cpu().numpy(), L, k, S, T, t_exp=t_exp,
                                   t_mean=t_mean, t_median=t_median)
    assert_results_equal(dgot, dref, "per-chunk thresholds, direct")
