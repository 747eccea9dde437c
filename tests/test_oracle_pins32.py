"""Pins of the oracle's 32-bit field variant (fp32 chunks committed over Z_q, q = 2^32 - 5) against
what the mathematics fixes: primality of q, inverses and polynomials checked with Python integers,
closed forms, the byte layout, and statistics predicted by hand.  No GPU, no CUDA code."""
import numpy as np
import pytest

import oracle

Q = 2 ** 32 - 5


def is_prime(n):
    if n % 2 == 0:
        return n == 2
    d = np.arange(3, int(n ** 0.5) + 2, 2, dtype=np.int64)
    return not (n % d == 0).any()


def test_q_is_the_largest_prime_below_2_32():
    assert oracle.Q_FIELD == Q
    assert is_prime(Q)
    assert not any(is_prime(n) for n in range(Q + 1, 2 ** 32))
    # every finite fp32 pattern and both infinities stay below q: only five NaN patterns do not
    assert 0xFF800000 < Q and 2 ** 32 - Q == 5


def test_inverse_against_python_integers():
    rng = np.random.default_rng(1)
    for a in [1, 2, 3, Q - 1, Q - 2, 65521, 2 ** 31] + rng.integers(1, Q, 500).tolist():
        inv = oracle.mod_inverse32(int(a))
        assert 0 < inv < Q and (int(a) * inv) % Q == 1
        assert oracle.mod_inverse_euclid(int(a), Q) == inv          # the extended Euclidean method gives the same element
    assert oracle.mod_inverse32(Q - 1) == Q - 1                     # -1 is its own inverse


def poly_eval(c, x):
    acc = 0
    for cd in reversed([int(v) for v in c]):
        acc = (acc * int(x) + cd) % Q
    return acc


def test_horner_against_python_integers():
    rng = np.random.default_rng(2)
    c = rng.integers(0, Q, 40).astype(np.uint32)
    for x in [0, 1, 2, 65535, Q - 1] + rng.integers(0, 65536, 20).tolist():
        assert oracle.horner32(c, int(x)) == poly_eval(c, x)
    assert oracle.horner32(np.array([7], np.uint32), 12345) == 7


def test_interpolation_hand_example_and_closed_forms():
    # -1 + 4x - x^2 through (1, 2), (2, 3), (4, -1)
    assert oracle.interpolate32([1, 2, 4], [2, 3, Q - 1]).tolist() == [Q - 1, 4, Q - 1]
    assert oracle.interpolate32([9], [1234567890]).tolist() == [1234567890]
    # two points: slope (y1 - y0) / (x1 - x0), intercept y0 - slope x0
    x0, y0, x1, y1 = 5, 4000000000, 300, 17
    slope = ((y1 - y0) * pow(x1 - x0, -1, Q)) % Q
    assert oracle.interpolate32([x0, x1], [y0, y1]).tolist() == [(y0 - slope * x0) % Q, slope]


@pytest.mark.parametrize("k", [1, 2, 7, 32, 128])
def test_interpolant_passes_through_every_point_and_both_methods_agree(k):
    rng = np.random.default_rng(10 + k)
    x = rng.choice(65536, size=k, replace=False).astype(np.uint32)
    y = rng.integers(0, Q, k).astype(np.uint32)
    c = oracle.interpolate32(x, y)
    assert c.dtype == np.uint32 and (c.astype(np.int64) < Q).all()
    for xj, yj in zip(x.tolist(), y.tolist()):
        assert poly_eval(c, xj) == yj
    assert oracle.interpolate32(x, y, lagrange=True).tolist() == c.tolist()


def test_interpolation_rejects_repeated_x():
    with pytest.raises(ValueError):
        oracle.interpolate32([3, 8, 3], [1, 2, 3])
    with pytest.raises(ValueError):
        oracle.interpolate32([3, 8, 3], [1, 2, 3], lagrange=True)


def test_encode_decode_layout():
    proof = oracle.encode32(65536, [0x01020304, Q - 1])
    assert proof.tolist() == [0, 0, 4, 3, 2, 1, 0xFA, 0xFF, 0xFF, 0xFF]       # 65536 -> 0; little-endian words
    assert oracle.decode32(proof)[:3] == (oracle.ST_OK, 2, 65536)
    assert oracle.decode32(oracle.encode32(40000, [5, 6, 7]))[1:3] == (3, 40000)
    st, k, m, c = oracle.decode32(oracle.encode32(32769, [5, 6, 7]))
    assert st == oracle.ST_OK and c.tolist() == [5, 6, 7]
    bad_coeff = proof.copy()
    bad_coeff[6:10] = [0xFB, 0xFF, 0xFF, 0xFF]                                # = q
    assert oracle.decode32(bad_coeff)[0] == oracle.ST_BAD_PROOF
    assert oracle.decode32(oracle.encode32(32768, [1]))[0] == oracle.ST_BAD_PROOF
    assert oracle.decode32(proof[:9])[0] == oracle.ST_BAD_PROOF               # not 2 + 4k bytes


def chunk_of(rng, rows, hidden):
    return (rng.standard_t(3, size=(rows, hidden)) * 0.5).astype(np.float32)


def brute_topk(patterns, k):
    flat = patterns.reshape(-1)
    key = (flat & 0x7FFFFFFF).astype(np.int64)
    order = np.lexsort((np.arange(flat.size), -key))[:k]
    return order.astype(np.uint32), flat[order]


@pytest.mark.parametrize("k", [8, 128])
def test_proof_commits_to_every_selected_pattern(k):
    rng = np.random.default_rng(20 + k)
    act = chunk_of(rng, 16, 512)
    proofs, status, indices = oracle.build_proofs(act, 16, k, 1, 16, wide=True, threads=1)
    assert proofs.shape == (1, 2 + 4 * k) and status.tolist() == [0]
    idx, pat = brute_topk(act.view(np.uint32), k)
    assert indices[0].tolist() == idx.tolist()
    st, kk, m, c = oracle.decode32(proofs[0])
    assert (st, kk, m) == (oracle.ST_OK, k, 65536)                           # all indices below 2^15 + 1
    for i, v in zip(idx.tolist(), pat.tolist()):
        assert poly_eval(c, i % m) == v % Q


def test_identical_activations_validate_with_zero_error_and_the_paper_thresholds():
    rng = np.random.default_rng(30)
    act = chunk_of(rng, 64, 256)
    proofs, _, idx = oracle.build_proofs(act, 32, 128, 1, 64, wide=True)
    res = oracle.verify_proofs(act, proofs, 32, 128, 1, 64, t_exp=8, t_mean=256.0, t_median=128.0,
                               gen_indices=idx, wide=True)
    assert res["accept"].tolist() == [1, 1] and res["n_match"].tolist() == [128, 128]
    assert not res["exp_mismatch"].any() and not res["mant_diff_sum"].any() and not res["topk_mismatch"].any()


def staircase(deltas_low_bits):
    """One chunk whose 8 largest magnitudes are 2^10 .. 2^3 (distinct exponents, zero mantissas)."""
    act = np.zeros((4, 64), np.float32)
    act[0, :8] = [1024.0, -512.0, 256.0, 128.0, 64.0, 32.0, 16.0, 8.0]
    return act


def test_mantissa_statistics_predicted_by_hand():
    act = staircase(None)
    proofs, status, _ = oracle.build_proofs(act, 4, 8, 1, 4, wide=True)
    assert status.tolist() == [0]
    seen = act.view(np.uint32).copy()
    deltas = [0, 1, 5, 300, 70000, 2 ** 23 - 1, 0, 0]          # added to the 23-bit mantissas
    for j, d in enumerate(deltas):
        seen[0, j] += d
    res = oracle.verify_proofs(seen.view(np.float32), proofs, 4, 8, 1, 4, t_exp=8, t_mean=1e9, t_median=1e9,
                               wide=True)[0]
    assert res["exp_mismatch"] == 0 and res["n_match"] == 8
    assert res["mant_diff_sum"] == sum(deltas) and res["mant_mean"] == sum(deltas) / 8
    assert res["mant_median"] == (1 + 5) / 2                    # sorted: 0 0 0 1 | 5 300 70000 8388607
    # an exponent change and a sign flip each cost one exponent mismatch; the flip only under that reading
    seen = act.view(np.uint32).copy()
    seen[0, 2] += 1 << 23
    seen[0, 3] ^= 1 << 31
    kw = dict(t_exp=8, t_mean=256.0, t_median=128.0, wide=True)
    assert oracle.verify_proofs(seen.view(np.float32), proofs, 4, 8, 1, 4, **kw)[0]["exp_mismatch"] == 2
    assert oracle.verify_proofs(seen.view(np.float32), proofs, 4, 8, 1, 4, sign_in_exponent=False,
                                **kw)[0]["exp_mismatch"] == 1


def test_thresholds_are_strict_and_nothing_matched_is_rejected():
    act = staircase(None)
    proofs, _, _ = oracle.build_proofs(act, 4, 8, 1, 4, wide=True)
    seen = act.view(np.uint32).copy()
    seen[0, :8] += 256                                          # every difference is exactly 256
    at = oracle.verify_proofs(seen.view(np.float32), proofs, 4, 8, 1, 4, t_exp=8, t_mean=256.0, t_median=256.0,
                              wide=True)[0]
    assert at["accept"] == 1 and at["mant_mean"] == 256.0 and at["mant_median"] == 256.0
    below = oracle.verify_proofs(seen.view(np.float32), proofs, 4, 8, 1, 4, t_exp=8, t_mean=255.5, t_median=256.0,
                                 wide=True)[0]
    assert below["accept"] == 0
    seen = act.view(np.uint32).copy()
    seen[0, :8] += 1 << 23                                      # every exponent differs
    none = oracle.verify_proofs(seen.view(np.float32), proofs, 4, 8, 1, 4, t_exp=100, t_mean=1e9, t_median=1e9,
                                wide=True)[0]
    assert none["n_match"] == 0 and none["accept"] == 0


def test_statuses():
    act = staircase(None)
    proofs, status, _ = oracle.build_proofs(act, 4, 8, 1, 4, wide=True)
    # a pattern >= q (a negative NaN with the largest payloads) is flagged, the proof still made
    nan = act.view(np.uint32).copy()
    nan[1, 5] = 0xFFFFFFFD
    p2, s2, _ = oracle.build_proofs(nan.view(np.float32), 4, 8, 1, 4, wide=True)
    assert s2.tolist() == [oracle.ST_NONFINITE] and p2.any()
    # fewer than k elements
    p3, s3, _ = oracle.build_proofs(act[:, :1].copy(), 4, 8, 1, 4, wide=True)
    assert s3.tolist() == [oracle.ST_K_EXCEEDS] and not p3.any()
    bad = proofs.copy()
    bad[0, 2:6] = [0xFF, 0xFF, 0xFF, 0xFF]
    res = oracle.verify_proofs(act, bad, 4, 8, 1, 4, wide=True)[0]
    assert res["status"] == oracle.ST_BAD_PROOF and res["accept"] == 0
    with pytest.raises(TypeError):
        oracle.build_proofs(np.zeros((4, 64), np.uint16), 4, 8, 1, 4, wide=True)


def test_wide_and_narrow_proofs_of_an_fp32_chunk_share_selection_and_modulus():
    rng = np.random.default_rng(40)
    act = chunk_of(rng, 32, 2048)
    wide, _, wi = oracle.build_proofs(act, 32, 128, 1, 32, wide=True)
    narrow, _, ni = oracle.build_proofs(act, 32, 128, 1, 32)
    assert wi.tolist() == ni.tolist() and wide[0, :2].tolist() == narrow[0, :2].tolist()
    assert wide.shape[1] == 2 + 4 * 128 and narrow.shape[1] == 2 + 2 * 128


def test_padded_validation_of_a_bf16_proof_against_fp32_activations():
    """Section 5.6: the committed 16-bit pattern is padded with 16 zero bits and compared with the fp32
    validator's pattern.  fp32 values whose upper halves are the generator's bf16 patterns differ from
    the padded commitment by exactly their lower 16 bits."""
    upper = np.zeros((4, 64), np.uint16)
    upper[0, :8] = [0x4480, 0xC400, 0x4380, 0x4300, 0x4280, 0x4200, 0x4180, 0x4100]    # 1024, -512, 256 .. 8
    low = np.zeros((4, 64), np.uint32)
    deltas = [0, 1, 77, 300, 20000, 0x7FFF, 5, 5]
    low[0, :8] = deltas
    fp32 = (upper.astype(np.uint32) << 16) | low
    proofs, status, idx = oracle.build_proofs(upper, 4, 8, 1, 4)                       # the bf16 generator
    assert status.tolist() == [0] and proofs.shape == (1, 2 + 2 * 8)
    res = oracle.verify_proofs(fp32.view(np.float32), proofs, 4, 8, 1, 4, t_exp=8, t_mean=1e9, t_median=1e9,
                               gen_indices=idx, padded=True)[0]
    assert res["exp_mismatch"] == 0 and res["n_match"] == 8 and res["topk_mismatch"] == 0
    assert res["mant_diff_sum"] == sum(deltas) and res["mant_mean"] == sum(deltas) / 8
    assert res["mant_median"] == (5 + 77) / 2 and res["accept"] == 1                   # 0 1 5 5 | 77 300 20000 32767
    strict = oracle.verify_proofs(fp32.view(np.float32), proofs, 4, 8, 1, 4, t_exp=8, t_mean=256.0,
                                  t_median=128.0, padded=True)[0]
    assert strict["accept"] == 0                                                       # the mean is far above 256
    exact = oracle.verify_proofs((upper.astype(np.uint32) << 16).view(np.float32), proofs, 4, 8, 1, 4, t_exp=8,
                                 t_mean=256.0, t_median=128.0, padded=True)[0]
    assert exact["accept"] == 1 and exact["mant_diff_sum"] == 0
    # an exponent change in the validator's value is an exponent mismatch, not a mantissa difference
    bumped = fp32.copy()
    bumped[0, 4] += 1 << 23
    assert oracle.verify_proofs(bumped.view(np.float32), proofs, 4, 8, 1, 4, t_exp=8, t_mean=1e9, t_median=1e9,
                                padded=True)[0]["exp_mismatch"] == 1
    with pytest.raises(TypeError):
        oracle.verify_proofs(upper, proofs, 4, 8, 1, 4, padded=True)
