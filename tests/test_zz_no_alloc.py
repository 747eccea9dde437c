"""The workspace-free entry point (collected last on purpose: a failure here must not hide
the results of any other test).

`toploc_build_proofs_builtin_scratch` serves embedders that cannot allocate device memory at
the point where proofs are generated -- an engine hook working inside a fixed memory pool, a
plug-in that only ever receives pointers.  Its scratch is a buffer inside the library.  The
test calls it through the C ABI twice in a row on different inputs and expects exactly what
the ordinary entry point and the CPU oracle produce (proof bytes, statuses and indices are
integers: equality, as everywhere in the parity tests), so a second call cannot be fooled by
what the first left in the shared buffer; it checks that the device's free memory does not
move across a call, and that oversized and ragged batches are refused.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_16007_b200 as tl
from paper_2501_16007_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def outputs(n, k):
    return (torch.zeros((n, 2 + 2 * k), dtype=torch.uint8, device=DEV),
            torch.full((n,), 255, dtype=torch.uint8, device=DEV),
            torch.full((n, k), -1, dtype=torch.int32, device=DEV))


def test_builtin_scratch_matches_the_workspace_entry_point_twice_in_a_row():
    cases = [  # (sequences, tokens, hidden, chunk_len, k, seed, recipe): the second is larger than the first
        (3, 96, 4096, 32, 128, 31, "jitter"),
        (6, 128, 2048, 16, 64, 32, "fixed"),
    ]
    for call, (S, T, H, L, k, seed, recipe) in enumerate(cases):
        act = synth.make_activations(S, T, H, torch.bfloat16, seed=seed, device=DEV, outliers=recipe)
        lay, _ = tl.make_layout(act, L, k, S, T)
        n = tl.toploc_num_chunks(lay)
        assert tl.toploc_workspace_bytes(lay) <= tl.TOPLOC_BUILTIN_SCRATCH_BYTES
        want = tl.toploc_build_proofs(act, lay, want_indices=True)
        got = outputs(n, k)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        tl.toploc_build_proofs_builtin_scratch(act, lay, *got)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        if call > 0:
            # (the first call of a process may load kernels and look the buffer's address up; from
            # the second call on, the device's free memory must not move at all)
            assert free_after == free_before, "the call changed the device's free memory"
        for g, w, name in zip(got, want, ("proofs", "status", "indices")):
            assert np.array_equal(g.cpu().numpy(), w.cpu().numpy()), "%s differ (S=%d)" % (name, S)
        assert not got[1].any().item()
        # and against the CPU oracle directly, not only through the other entry point
        ref = oracle.build_proofs(synth.host_patterns(act), L, k, S, T)
        for g, r, name in zip(got, ref, ("proofs", "status", "indices")):
            assert np.array_equal(g.cpu().numpy(), r), "%s differ from the oracle (S=%d)" % (name, S)


def test_builtin_scratch_refuses_what_does_not_fit():
    act = torch.zeros((64, 64), dtype=torch.bfloat16, device=DEV)
    lay, _ = tl.make_layout(act, 32, 8, 2, 32)
    lay.num_seqs, lay.tokens_per_seq, lay.k = 4096, 4096, 128      # 524288 chunks: far beyond 8 MiB
    assert tl.toploc_workspace_bytes(lay) > tl.TOPLOC_BUILTIN_SCRATCH_BYTES
    n_small = 4
    with pytest.raises(tl.ToplocError, match="built-in"):
        tl.toploc_build_proofs_builtin_scratch(act, lay, *outputs(n_small, 128))
    ragged, keep = tl.make_layout(act, 32, 8, 2, seq_offsets=[0, 30, 64])
    with pytest.raises(tl.ToplocError, match="unsupported"):
        tl.toploc_build_proofs_builtin_scratch(act, ragged, *outputs(2, 8))
