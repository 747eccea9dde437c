"""Pins of the oracle's direct commitments (Section 4: top-k indices and values stored as they
are, 6 bytes per point) to things other than itself: numpy's own ordering, hand-built
commitments whose statistics are predicted by hand, and the already pinned polynomial path,
whose validation must give the same statistics whenever both sides select the same indices.
Nothing here touches the CUDA library."""
import numpy as np
import pytest
import torch

import oracle
from paper_2501_16007_b200 import synth


def bf16_bits(values):
    t = torch.tensor(values, dtype=torch.float32).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def records(commit):
    """Independent decoder of the 6-byte records."""
    rec = np.asarray(commit, np.uint8).reshape(-1, 6).astype(np.uint32)
    idx = rec[:, 0] | (rec[:, 1] << 8) | (rec[:, 2] << 16) | (rec[:, 3] << 24)
    bits = (rec[:, 4] | (rec[:, 5] << 8)).astype(np.uint16)
    return idx, bits


def make_commit(idx, bits):
    out = np.zeros((len(idx), 6), np.uint8)
    for j, (i, b) in enumerate(zip(idx, bits)):
        out[j] = [i & 255, (i >> 8) & 255, (i >> 16) & 255, (i >> 24) & 255, b & 255, (b >> 8) & 255]
    return out.reshape(1, -1)


def numpy_topk_set(chunk, k):
    """Top-k by (magnitude key descending, flat index ascending) stated with numpy's lexsort."""
    flat = chunk.reshape(-1)
    key = (flat & 0x7FFF).astype(np.int64) if flat.dtype == np.uint16 else (flat & 0x7FFFFFFF).astype(np.int64)
    order = np.lexsort((np.arange(flat.size), -key))
    return np.sort(order[:k])


def test_storage_is_six_bytes_per_point():
    a = np.arange(1, 257, dtype=np.uint16).reshape(4, 64)
    for k in (1, 7, 128):
        commits, status = oracle.commit_direct(a, 4, k, 1, 4)
        assert commits.shape == (1, 6 * k) and status[0] == oracle.ST_OK
    # Section 4: three times the 2 bytes per point of a coefficient
    assert 6 * 128 == 3 * (258 - 2)


@pytest.mark.parametrize("k", [1, 5, 64, 600, 4096])
def test_records_are_the_topk_in_index_order(k):
    rng = np.random.default_rng(k)
    # few distinct magnitudes: the cut falls inside a run of ties
    a = rng.integers(0x3F00, 0x3F40, size=(16, 512), dtype=np.uint16)
    a ^= (rng.integers(0, 2, size=a.shape, dtype=np.uint16) << 15)
    commits, status = oracle.commit_direct(a, 16, k, 1, 16)
    assert status[0] == oracle.ST_OK
    idx, bits = records(commits[0])
    assert np.array_equal(idx, numpy_topk_set(a, k))
    assert np.array_equal(bits, a.reshape(-1)[idx])


def test_fp32_ranks_on_all_bits_and_commits_the_upper_half():
    rng = np.random.default_rng(3)
    a = rng.standard_normal((4, 256)).astype(np.float32)
    a[1, 7] = a[2, 9] = 5.0                      # equal upper halves, ordered by the lower bits
    u = a.view(np.uint32).copy()
    u[2, 9] += 1
    commits, status = oracle.commit_direct(u, 4, 1, 1, 4)
    idx, bits = records(commits[0])
    assert idx[0] == 2 * 256 + 9 and bits[0] == (u[2, 9] >> 16)
    commits, _ = oracle.commit_direct(u, 4, 40, 1, 4)
    idx, bits = records(commits[0])
    assert np.array_equal(idx, numpy_topk_set(u, 40))
    assert np.array_equal(bits, (u.reshape(-1)[idx] >> 16).astype(np.uint16))


def test_identical_activations_validate_with_zero_statistics():
    act = synth.make_activations(1, 64, 512, torch.bfloat16, seed=5)
    host = synth.host_patterns(act)
    for k in (128, 1024):
        commits, status = oracle.commit_direct(host, 32, k, 1, 64)
        res, dev = oracle.verify_direct(host, commits, 32, k, 1, 64, t_exp=38 * k // 128)
        assert (res["status"] == 0).all() and (res["accept"] == 1).all()
        assert (res["exp_mismatch"] == 0).all() and (res["n_match"] == k).all()
        assert (res["mant_diff_sum"] == 0).all() and (res["topk_mismatch"] == 0).all()
        assert (dev[:, 0] == k).all() and (dev[:, 1:] == 0).all()


def test_same_statistics_as_the_polynomial_when_the_index_sets_agree():
    """P(x_j) = y_j at every committed index, so looking a committed index up and evaluating the
    polynomial there are the same thing; the two validations can only differ at indices that
    were not committed."""
    # one sequence with outlier channels (the +1-ulp copy keeps its index sets) and one of plain
    # heavy-tailed data (many values near the cut: the copy moves some indices in and out)
    act = torch.cat([synth.make_activations(1, 128, 1024, torch.bfloat16, seed=11, outliers="jitter"),
                     synth.make_activations(1, 128, 1024, torch.bfloat16, seed=13, outliers="none")])
    noisy = synth.plus_one_ulp(act, seed=12)
    host, rec = synth.host_patterns(act), synth.host_patterns(noisy)
    k = 128
    proofs, st, gen_idx = oracle.build_proofs(host, 32, k, 2, 128)
    poly = oracle.verify_proofs(rec, proofs, 32, k, 2, 128, gen_indices=gen_idx)
    commits, st2 = oracle.commit_direct(host, 32, k, 2, 128)
    direct, _ = oracle.verify_direct(rec, commits, 32, k, 2, 128)
    same = poly["topk_mismatch"] == 0
    assert same.any() and (poly["topk_mismatch"] > 0).any()      # both kinds of chunk occur
    for f in ("exp_mismatch", "n_match", "mant_diff_sum", "mant_mean", "mant_median", "accept", "topk_mismatch"):
        assert np.array_equal(poly[f][same], direct[f][same]), f
    # where the sets differ, every uncommitted index is a mismatch in the direct form
    assert (direct["exp_mismatch"] >= direct["topk_mismatch"]).all()
    assert np.array_equal(poly["topk_mismatch"], direct["topk_mismatch"])


def test_hand_built_statistics_and_deviation_bins():
    # eight elements, k = 4; the validator's top-4 are flat indices 0, 1, 2, 3
    seen = bf16_bits([8.0, 4.0, -2.0, 1.0, 0.1, 0.1, 0.1, 0.1]).reshape(1, 8)
    e = lambda v: int(bf16_bits([v])[0])
    # committed: index 0 with the same exponent and mantissa + 3; index 1 with the exponent one
    # higher (seen - committed = -1); index 2 with the sign flipped; index 5 instead of index 3
    commit = make_commit([0, 1, 2, 5], [e(8.0) + 3, e(8.0), e(2.0), e(0.1)])
    res, dev = oracle.verify_direct(seen, commit, 1, 4, 1, 1, t_exp=4, t_mean=10, t_median=8)
    r = res[0]
    assert r["status"] == 0 and r["topk_mismatch"] == 1
    assert r["exp_mismatch"] == 3            # higher exponent, flipped sign, uncommitted index
    assert r["n_match"] == 1 and r["mant_diff_sum"] == 3 and r["mant_mean"] == 3.0 and r["mant_median"] == 3.0
    assert r["accept"] == 1
    assert dev[0].tolist() == [2, 1, 0, 0, 0, 0, 0, 0, 0]   # the sign is not part of the deviation
    res, _ = oracle.verify_direct(seen, commit, 1, 4, 1, 1, t_exp=2, t_mean=10, t_median=8)
    assert res[0]["accept"] == 0             # 3 > 2, strict comparison as in Algorithm 2
    res, dev = oracle.verify_direct(seen, commit, 1, 4, 1, 1, t_exp=4, sign_in_exponent=False)
    assert res[0]["exp_mismatch"] == 2 and res[0]["n_match"] == 2


def test_deviation_bins_cover_every_distance():
    for d, want in [(0, 0), (-1, 1), (1, 2), (-2, 3), (2, 4), (-3, 5), (-10, 5), (3, 6), (10, 6), (11, 7),
                    (-11, 7), (99, 7), (-99, 7), (100, 8), (-100, 8), (120, 8)]:
        committed_exp = 127 if d <= 0 else 1
        seen_exp = committed_exp + d
        assert 0 < seen_exp < 255
        seen = np.array([[seen_exp << 7, 0]], np.uint16)
        commit = make_commit([0], [committed_exp << 7])
        _, dev = oracle.verify_direct(seen, commit, 1, 1, 1, 1)
        assert dev[0].sum() == 1 and dev[0][want] == 1, (d, dev[0])


def test_median_of_an_even_count_and_strict_thresholds():
    seen = bf16_bits([8.0, 8.0, 8.0, 8.0]).reshape(1, 4)
    base = int(seen[0, 0])
    commit = make_commit([0, 1, 2, 3], [base + 1, base + 2, base + 9, base + 20])
    res, _ = oracle.verify_direct(seen, commit, 1, 4, 1, 1, t_exp=0, t_mean=8.0, t_median=5.5)
    r = res[0]
    assert r["mant_diff_sum"] == 32 and r["mant_mean"] == 8.0 and r["mant_median"] == 5.5 and r["accept"] == 1
    res, _ = oracle.verify_direct(seen, commit, 1, 4, 1, 1, t_exp=0, t_mean=7.99, t_median=5.5)
    assert res[0]["accept"] == 0
    res, _ = oracle.verify_direct(seen, commit, 1, 4, 1, 1, t_exp=0, t_mean=8.0, t_median=5.0)
    assert res[0]["accept"] == 0


def test_malformed_commitments_and_short_chunks():
    seen = bf16_bits([4.0, 3.0, 2.0, 1.0]).reshape(1, 4)
    ok = make_commit([0, 1], [int(seen[0, 0]), int(seen[0, 1])])
    assert oracle.verify_direct(seen, ok, 1, 2, 1, 1)[0][0]["status"] == oracle.ST_OK
    for idx in ([1, 0], [1, 1], [0, 4], [0, 2 ** 31]):
        bad = make_commit(idx, [0, 0])
        r = oracle.verify_direct(seen, bad, 1, 2, 1, 1)[0][0]
        assert r["status"] == oracle.ST_BAD_PROOF and r["accept"] == 0, idx
    commits, status = oracle.commit_direct(seen, 1, 5, 1, 1)
    assert status[0] == oracle.ST_K_EXCEEDS and not commits.any()
    r = oracle.verify_direct(seen, commits, 1, 5, 1, 1)[0][0]
    assert r["status"] == oracle.ST_K_EXCEEDS and r["accept"] == 0


def test_tampering_is_rejected_and_noise_accepted_at_large_k():
    k = 1024
    act = synth.make_activations(1, 64, 2048, torch.bfloat16, seed=21, outliers="none")
    host = synth.host_patterns(act)
    commits, _ = oracle.commit_direct(host, 32, k, 1, 64)
    other = synth.host_patterns(synth.make_activations(1, 64, 2048, torch.bfloat16, seed=22, outliers="none"))
    res, _ = oracle.verify_direct(other, commits, 32, k, 1, 64, t_exp=38 * k // 128)
    assert (res["accept"] == 0).all()
    trunc = synth.host_patterns(synth.truncate_mantissa(act, 1))
    res, _ = oracle.verify_direct(trunc, commits, 32, k, 1, 64, t_exp=38 * k // 128)
    assert (res["accept"] == 0).all()
