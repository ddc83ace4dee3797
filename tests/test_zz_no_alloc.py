"""The allocation-free greedy acceptance entry point against the regular one.

Some callers of this library may not allocate device memory (all of it belongs to their framework's
pool, or they sit in a loop where an allocating call is forbidden).  For them as_accept_greedy_static
keeps its scratch in a fixed array inside the library.  This test calls it through the C ABI twice in a
row, with different inputs, and requires bit-identical results to the CPU oracle's greedy acceptance and to
as_accept (which uses a caller-bound workspace).  The second call starts from whatever the first one left in the shared array, so it also
checks that the call clears what it must.  The file sorts last so that a run stopping at the first
failure has already executed every other test."""
import numpy as np
import pytest
import torch

from paper_2608_24004_b200 import workloads
from helpers import oracle_accept

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bnd():
    from paper_2608_24004_b200 import build as as_build
    as_build.build_library()
    from paper_2608_24004_b200 import binding
    return binding


def _both(bnd, b):
    vs = bnd.VerifyStep(b)
    vs.plan_step()
    vs.accept()                                            # reference: plan + workspace
    assert bnd.as_plan_check(vs.plan) == 0
    cu_q = torch.as_tensor(np.concatenate([[0], np.cumsum(b.draft_lens + 1)]).astype(np.int32)).cuda()
    acc = torch.full((b.batch,), -7, dtype=torch.int32, device="cuda")
    toks = torch.full((b.batch, b.k_max + 1), -7, dtype=torch.int32, device="cuda")
    bnd.as_accept_greedy_static(b.batch, b.total_q, b.k_max, cu_q, vs.logits, b.vocab, vs.draft_tokens, acc, toks)
    torch.cuda.synchronize()
    assert torch.equal(acc, vs.accept_len), (acc, vs.accept_len)
    assert torch.equal(toks, vs.out_tokens)
    ref = oracle_accept(b)                                 # and the oracle itself, not only the other CUDA path
    assert np.array_equal(acc.cpu().numpy(), ref["accept_len"])
    assert np.array_equal(toks.cpu().numpy(), ref["out_tokens"])
    return int(acc.sum())


def test_static_scratch_entry_point_matches_as_accept_twice_in_a_row(bnd):
    first = workloads.make_batch("a", seed=31, seq_lens=[20] * 40, draft_lens=list(np.arange(40) % 9), num_q_heads=8,
                                 num_kv_heads=2, head_dim=128, vocab=151936, logit_std=2.0, match_p=0.7, k_max=8)
    first.logits[0, :] = 1.0                               # an all-ties row: lowest index must win
    first.logits[1, 5] = float("nan")
    second = workloads.make_batch("b", seed=32, seq_lens=[20] * 17, draft_lens=[8] * 10 + [0] * 7, num_q_heads=8,
                                  num_kv_heads=2, head_dim=128, vocab=5001, ld=5004, logit_std=2.0, match_p=0.9,
                                  k_max=8)
    accepted = _both(bnd, first) + _both(bnd, second)      # second call reuses the array the first one filled
    assert accepted > 20


def test_static_scratch_entry_point_rejects_oversized_batches(bnd):
    rows = bnd.AS_STATIC_MAX_ROWS + 1
    z = torch.zeros((4, 8), dtype=torch.float32, device="cuda")
    dummy = torch.zeros(rows + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(bnd.AsError) as e:
        bnd.as_accept_greedy_static(rows, rows, 0, dummy, z, 8, None, dummy, dummy)
    assert e.value.status == bnd.AS_ERR_INVALID_ARG and "AS_STATIC_MAX_ROWS" in str(e.value)


def test_static_scratch_entry_point_survives_a_malformed_cu_q(bnd):
    """cu_q lives in device memory, so the entry point cannot check it before launching.  Entries that run backwards,
    promise more drafts than max_draft or point past total_q must cost their own request its result (accept_len 0, a
    row of -1) and nothing else: no fault, the other requests exact, free device memory unchanged by the call."""
    b = workloads.make_batch("c", seed=33, seq_lens=[20] * 6, draft_lens=[4, 2, 0, 4, 3, 1], num_q_heads=8, num_kv_heads=2,
                             head_dim=128, vocab=777, logit_std=2.0, match_p=0.8, k_max=4)
    ref = oracle_accept(b)
    good = np.concatenate([[0], np.cumsum(b.draft_lens + 1)]).astype(np.int32)
    logits = b.logits.cuda()
    drafts = torch.as_tensor(b.draft_tokens).cuda()
    for bad_req, entry, value in [(1, 2, 3), (3, 4, 100000), (0, 1, 9), (4, 5, -6)]:
        cu_q = good.copy()
        cu_q[entry] = value
        broken = {i for i in range(b.batch) if not (cu_q[i] >= i and 0 <= cu_q[i + 1] - cu_q[i] - 1 <= b.k_max
                                                    and cu_q[i + 1] - 1 < b.total_q)}
        assert bad_req in broken
        acc = torch.full((b.batch,), -7, dtype=torch.int32, device="cuda")
        toks = torch.full((b.batch, b.k_max + 1), -7, dtype=torch.int32, device="cuda")
        free_before = torch.cuda.mem_get_info()[0]
        bnd.as_accept_greedy_static(b.batch, b.total_q, b.k_max, torch.as_tensor(cu_q).cuda(), logits, b.vocab, drafts, acc, toks)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] >= free_before - (1 << 20)
        acc, toks = acc.cpu().numpy(), toks.cpu().numpy()
        for i in range(b.batch):
            if i in broken:
                assert acc[i] == 0 and (toks[i] == -1).all()
            elif cu_q[i] == good[i] and cu_q[i + 1] == good[i + 1]:
                assert acc[i] == ref["accept_len"][i] and np.array_equal(toks[i], ref["out_tokens"][i])
