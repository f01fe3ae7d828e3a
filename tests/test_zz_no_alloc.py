"""specvlm_accept_noalloc: the acceptance step for callers that cannot allocate device memory
(a plug-in inside someone else's memory plan, a serving loop that must not call cudaMalloc) and
have no workspace to pass.  Its scratch is a fixed array inside the library, so the thing to
check is that it gives exactly what specvlm_accept gives (and what the CPU oracle gives) -- also
on a second call, when the array still holds the first call's candidates -- and that it refuses
problems larger than the array.  Collected last on purpose: a failure here cannot hide any other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_16201_b200 import specvlm, synth

pytestmark = pytest.mark.gpu


def _both(batch, gamma, vocab, seed):
    logits, drafts = synth.logits_and_drafts(batch, gamma, vocab, "cuda", seed)
    ref_n, ref_next, ref_g = specvlm.accept(logits, drafts, want_argmax=True)
    n = torch.full((batch,), -7, dtype=torch.int32, device="cuda")
    nxt = torch.full((batch,), -7, dtype=torch.int32, device="cuda")
    g = torch.full((batch, gamma + 1), -7, dtype=torch.int32, device="cuda")
    specvlm.accept_noalloc(logits, drafts, (n, nxt), want_argmax_into=g)
    torch.cuda.synchronize()
    # integer results: the tolerance of the other acceptance tests is bit-exactness
    assert torch.equal(n, ref_n) and torch.equal(nxt, ref_next) and torch.equal(g, ref_g)
    # and against the CPU oracle on the same logits and drafts, so that a defect shared by the two
    # CUDA entry points cannot pass
    lg, dr = logits.cpu().numpy(), drafts.cpu().numpy()
    for b in range(batch):
        on, onext, og = oracle.accept_fast(lg[b], dr[b])
        assert (int(n[b]), int(nxt[b])) == (on, onext) and np.array_equal(g[b].cpu().numpy(), og)


def test_noalloc_matches_accept_on_two_calls_in_a_row():
    # second call: a different, smaller problem, so stale candidates of the first call sit right
    # behind the slots it uses
    _both(16, 8, 152064, seed=31)
    _both(3, 5, 4099, seed=32)
    _both(16, 8, 152064, seed=33)


def test_noalloc_rejects_oversized_problem_and_bad_arguments():
    logits = torch.zeros((1, 2, 8), dtype=torch.float32, device="cuda")
    L = specvlm.lib()
    # 128 * 9 * ceil(152064 / 8192) = 21888 candidates > 16384: refused before any launch
    rc = L.specvlm_accept_noalloc(logits.data_ptr(), logits.data_ptr(), 128, 8, 152064, logits.data_ptr(),
                                  logits.data_ptr(), None, None)
    assert rc == specvlm.ERR_TOO_LARGE
    assert "built-in scratch" in specvlm.status_string(rc)
    rc = L.specvlm_accept_noalloc(None, None, 1, 1, 8, None, None, None, None)
    assert rc == specvlm.ERR_INVALID_ARG
