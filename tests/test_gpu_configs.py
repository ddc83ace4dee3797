"""GPU parity at the full sizes of the named workloads, in the launch configuration bench.py times.

Attention is compared on every request of the bench workload and on at least sixteen (eight at the sweep points)
of the others - always the shortest, the longest, the longest and the shortest draft - with all rows and heads of
each, which the oracle computes in seconds from a compact copy of just their pages; acceptance and commit are
compared in full.  Tolerances as in test_gpu_parity.py."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_24004_b200 import workloads
from helpers import oracle_attn, oracle_accept, oracle_commit, sub_batch, attn_errors, cu
from test_gpu_parity import bnd, check_attn, _check_sampled   # noqa: F401  (fixture + shared rules)

pytestmark = pytest.mark.gpu


def _sample_requests(b, count, rng):
    order = np.argsort(b.seq_lens)
    picks = {int(order[0]), int(order[-1]), int(np.argmax(b.draft_lens)), int(np.argmin(b.draft_lens))}
    while len(picks) < min(count, b.batch):
        picks.add(int(rng.integers(0, b.batch)))
    return sorted(picks)


def _attn_on_samples(bnd, b, vs, kind, req_ids):
    sb, rows = sub_batch(b, req_ids)
    want, want_lse = oracle_attn(sb, kind=kind)
    rows_t = torch.as_tensor(rows, device="cuda")
    check_attn(vs.out[kind][rows_t], vs.lse[kind][rows_t], want, want_lse)


def test_qwen3_8b_full_step(bnd):
    b = workloads.qwen3_8b(device="cuda")
    assert b.batch == 64 and b.seq_lens.min() >= 512 and b.seq_lens.max() <= 32768
    vs = bnd.VerifyStep(b)
    vs.plan_step(); vs.attn(0); vs.accept()
    assert bnd.as_plan_check(vs.plan) == 0
    _attn_on_samples(bnd, b, vs, 0, list(range(b.batch)))            # all 64 requests
    ref = oracle_accept(b)
    assert np.array_equal(vs.accept_len.cpu().numpy(), ref["accept_len"])
    assert np.array_equal(vs.out_tokens.cpu().numpy(), ref["out_tokens"])
    # generator sanity: drafts match the target argmax with probability 0.6, so E[a] = mean_k 1.5 (1 - 0.6^k)
    want = np.mean([1.5 * (1 - 0.6 ** k) for k in b.draft_lens])
    assert abs(ref["accept_len"].mean() - want) < 0.5
    vs.commit()
    assert bnd.as_plan_check(vs.plan) == 0
    a = ref["accept_len"]
    n_new = b.seq_lens + a + 1
    assert np.array_equal(vs.seq_lens.cpu().numpy(), n_new)
    bt = vs.block_table.cpu().numpy()
    keep = -(-n_new // b.block_size)
    freed_want = []
    for i in range(b.batch):
        assert (bt[i, keep[i]:] == -1).all() and np.array_equal(bt[i, :keep[i]], b.block_table[i, :keep[i]])
        freed_want += [int(x) for x in b.block_table[i, keep[i]:] if x >= 0]
    assert list(vs.freed.cpu().numpy()[:int(vs.freed_count.item())]) == freed_want


@pytest.mark.parametrize("all_max", [False, True])
def test_gpt_oss_20b_layer_pair(bnd, all_max):
    b = workloads.gpt_oss_20b(device="cuda", batch=128 if not all_max else 32, all_max=all_max)
    vs = bnd.VerifyStep(b)
    vs.plan_step(); vs.attn(0); vs.attn(1); vs.accept()
    assert bnd.as_plan_check(vs.plan) == 0
    ids = _sample_requests(b, 16, np.random.default_rng(1))
    _attn_on_samples(bnd, b, vs, 0, ids)
    _attn_on_samples(bnd, b, vs, 1, ids)
    ref = oracle_accept(b)
    assert np.array_equal(vs.accept_len.cpu().numpy(), ref["accept_len"])
    assert np.array_equal(vs.out_tokens.cpu().numpy(), ref["out_tokens"])


def test_r1_distill_llama_8b_stochastic(bnd):
    b = workloads.r1_distill_llama_8b(device="cuda")
    assert b.batch == 256 and b.draft_probs is not None
    vs = bnd.VerifyStep(b)
    vs.plan_step(); vs.attn(0); vs.accept()
    assert bnd.as_plan_check(vs.plan) == 0
    _attn_on_samples(bnd, b, vs, 0, _sample_requests(b, 16, np.random.default_rng(2)))
    in_band, total, exact = _check_sampled(bnd, b, vs)
    assert in_band < max(1, 1e-4 * total), (in_band, total)
    assert exact >= 0.99 * b.batch, exact


@pytest.mark.parametrize("batch,k,ctx", [(1, 16, 131072), (8, 4, 8192), (32, 1, 1024), (128, 8, 8192), (8, 0, 32768)])
def test_sweep_points(bnd, batch, k, ctx):
    b = workloads.sweep_point(batch, k, ctx, device="cuda")
    vs = bnd.VerifyStep(b)
    vs.plan_step(); vs.attn(0)
    assert bnd.as_plan_check(vs.plan) == 0
    _attn_on_samples(bnd, b, vs, 0, _sample_requests(b, 8, np.random.default_rng(3)))
