"""Shared plumbing of the GPU parity tests: run the CUDA path through the C ABI and the
oracle on the same bytes, and compare field by field."""
import numpy as np
import torch

import oracle
import paper_2501_16007_b200 as tl
from paper_2501_16007_b200 import synth

MEAN_TOL = 1e-9  # fp64 mean / median: absolute tolerance; every integer field is exact


def gpu_build(act, chunk_len, k, num_seqs, tokens_per_seq=0, seq_offsets=None, field=0):
    lay, keep = tl.make_layout(act, chunk_len, k, num_seqs, tokens_per_seq, seq_offsets, field=field)
    proofs, status, indices = tl.toploc_build_proofs(act, lay, want_indices=True)
    torch.cuda.synchronize()
    return proofs, status, indices


def gpu_verify(act, proofs, chunk_len, k, num_seqs, tokens_per_seq=0, seq_offsets=None, thresholds=None,
               gen_indices=None, field=0):
    lay, keep = tl.make_layout(act, chunk_len, k, num_seqs, tokens_per_seq, seq_offsets, field=field)
    thr = thresholds if thresholds is not None else tl.default_thresholds(k, field=field)
    res = tl.toploc_verify_proofs(act, lay, proofs, thr, gen_indices=gen_indices)
    torch.cuda.synchronize()
    return res.cpu().numpy().view(tl.RESULT_DTYPE).reshape(-1)


def oracle_thresholds(k, sign_in_exponent=True, wide=False):
    """Section 5.2: 38 / 10 / 8 for bf16, 8 / 256 / 128 for fp32 inference (the 32-bit field)."""
    if wide:
        return dict(t_exp=(8 * k) // 128, t_mean=256.0, t_median=128.0, sign_in_exponent=sign_in_exponent)
    return dict(t_exp=(38 * k) // 128, t_mean=10.0, t_median=8.0, sign_in_exponent=sign_in_exponent)


def assert_build_equal(gpu, ref, where=""):
    gp, gs, gi = gpu
    rp, rs, ri = ref
    gp, gs = gp.cpu().numpy(), gs.cpu().numpy()
    bad = np.nonzero(gs != rs)[0]
    assert bad.size == 0, "%s status differs at chunks %s" % (where, bad[:8])
    if gi is not None and ri is not None:
        gi = gi.cpu().numpy()
        bad = np.nonzero((gi != ri).any(axis=1))[0]
        assert bad.size == 0, "%s selected indices differ at chunks %s" % (where, bad[:8])
    bad = np.nonzero((gp != rp).any(axis=1))[0]
    assert bad.size == 0, "%s proof bytes differ at chunks %s" % (where, bad[:8])


def assert_results_equal(gpu, ref, where=""):
    for f in ("exp_mismatch", "n_match", "mant_diff_sum", "topk_mismatch", "modulus", "accept", "status"):
        bad = np.nonzero(gpu[f] != ref[f])[0]
        assert bad.size == 0, "%s %s differs at chunks %s: gpu %s oracle %s" % (
            where, f, bad[:8], gpu[f][bad[:8]], ref[f][bad[:8]])
    for f in ("mant_mean", "mant_median"):
        err = np.abs(gpu[f] - ref[f])
        assert (err <= MEAN_TOL).all(), "%s %s off by %g" % (where, f, err.max())


def parity_case(act, chunk_len, k, num_seqs, tokens_per_seq=0, seq_offsets=None, recomputed=None, where="",
                wide=False):
    """Build on both sides, compare; verify `recomputed` (default: the same activations plus any
    extra tensors given as a dict) on both sides, compare.  Returns the oracle's results."""
    host = synth.host_patterns(act) if act.is_contiguous() else None
    if host is None:
        # strided view: the oracle gets the same strided bytes through a numpy view
        base = synth.host_patterns(act._base)
        host = base[:, :act.shape[1]]
    field = tl.TOPLOC_FIELD_32 if wide else tl.TOPLOC_FIELD_16
    g = gpu_build(act, chunk_len, k, num_seqs, tokens_per_seq, seq_offsets, field=field)
    r = oracle.build_proofs(host, chunk_len, k, num_seqs, tokens_per_seq, seq_offsets, wide=wide)
    assert_build_equal(g, r, where + " build")
    out = {}
    cases = {"same": act}
    cases.update(recomputed or {})
    for name, rec in cases.items():
        rec_host = synth.host_patterns(rec) if rec.is_contiguous() else synth.host_patterns(rec._base)[:, :rec.shape[1]]
        gv = gpu_verify(rec, g[0], chunk_len, k, num_seqs, tokens_per_seq, seq_offsets, gen_indices=g[2],
                        field=field)
        rv = oracle.verify_proofs(rec_host, r[0], chunk_len, k, num_seqs, tokens_per_seq, seq_offsets,
                                  gen_indices=r[2], wide=wide, **oracle_thresholds(k, wide=wide))
        assert_results_equal(gv, rv, "%s verify[%s]" % (where, name))
        out[name] = rv
    return r, out
