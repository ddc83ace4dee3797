"""as_plan_device(): the step's metadata built by a kernel from device-resident length arrays.  Its work list
must be the host planner's, so every result of a step planned on the device equals, bit for bit, the result
of the same step planned on the host; a recorded step (plan + attention + acceptance + commit in one CUDA
graph) must replay for step after step while the lengths evolve on the device."""
import copy

import numpy as np
import pytest
import torch

from paper_2608_24004_b200 import workloads
from helpers import attn_errors, oracle_accept, oracle_attn

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bnd():
    from paper_2608_24004_b200 import build as as_build
    as_build.build_library()
    from paper_2608_24004_b200 import binding
    return binding


def _batch(seed, D, Hq, Hkv, window, B, kmax, vocab=500, long_ctx=False):
    rng = np.random.default_rng(seed)
    hi = 40000 if long_ctx else 3000
    seq = [int(rng.choice([0, 1, 15, 16, 17, 127, 128, 129, 255, 256])) if rng.random() < 0.3 else int(rng.integers(0, hi))
           for _ in range(B)]
    dl = [int(rng.integers(0, kmax + 1)) for _ in range(B)]
    dl[int(rng.integers(0, B))] = kmax
    kinds = [workloads.LayerKind(window=window, sinks=None)]
    return workloads.make_batch("pd", seed=seed, seq_lens=seq, draft_lens=dl, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D,
                                vocab=vocab, logit_std=2.0, match="iid", match_p=0.6, k_max=kmax, kinds=kinds)


CASES = [
    # (seed, D, Hq, Hkv, window, B, kmax, impl, long contexts)
    (1, 128, 32, 8, 0, 9, 8, "tc", False),
    (2, 128, 16, 4, 200, 7, 5, "tc", False),
    (3, 64, 64, 8, 0, 6, 16, "tc", False),          # rows-on-M kernel, two row blocks for the longest draft
    (4, 64, 64, 8, 128, 12, 9, "tc", True),
    (5, 128, 8, 2, 0, 5, 4, "simt", False),
    (6, 128, 32, 8, 0, 3, 6, "tc", True),           # few long requests: every pair is cut into many pieces
    (7, 128, 4, 4, 0, 1, 0, "tc", False),           # a single request without drafts
    (8, 128, 32, 8, 0, 300, 3, "tc", False),        # 2400 (request, kv-head) pairs: three chunks of the planner CTA
    (9, 64, 16, 2, 0, 1500, 1, "tc", False),        # 1500 requests: two chunks of requests, three of pairs
    (10, 128, 64, 8, 0, 7, 16, "tc", False),        # head_dim 128, up to 136 rows: requests cut into two row blocks
    (11, 128, 32, 4, 150, 5, 31, "tc", True),       # 256 rows: two full row blocks, long contexts, a window
    (12, 128, 24, 8, 0, 6, 60, "tc", False),        # three query heads per kv head: blocks of 42 positions (126 rows)
]


@pytest.mark.parametrize("case", CASES)
def test_step_planned_on_the_device_equals_step_planned_on_the_host(bnd, case):
    seed, D, Hq, Hkv, window, B, kmax, impl_name, long_ctx = case
    impl = bnd.AS_ATTN_TC if impl_name == "tc" else bnd.AS_ATTN_SIMT
    A = _batch(seed, D, Hq, Hkv, window, B, kmax, long_ctx=long_ctx)
    host, dev = bnd.VerifyStep(A, attn_impl=impl), bnd.VerifyStep(A, attn_impl=impl)
    for s in (host, dev):
        bnd.as_plan_set_fixed_launch(s.plan, True)
    dl_dev = torch.as_tensor(A.draft_lens, dtype=torch.int32, device="cuda")
    host.plan_step(); host.attn(0); host.accept(); host.commit()
    dev.plan_step_device(B, dl_dev); dev.attn(0); dev.accept(); dev.commit()
    torch.cuda.synchronize()
    assert bnd.as_plan_check(host.plan) == 0 and bnd.as_plan_check(dev.plan) == 0
    tq = A.total_q
    assert torch.equal(dev.out[0][:tq], host.out[0][:tq]) and torch.equal(dev.lse[0][:tq], host.lse[0][:tq])
    assert torch.equal(dev.accept_len[:B], host.accept_len[:B]) and torch.equal(dev.out_tokens[:B], host.out_tokens[:B])
    assert torch.equal(dev.seq_lens, host.seq_lens) and torch.equal(dev.block_table, host.block_table)
    assert int(dev.freed_count.item()) == int(host.freed_count.item())
    nf = int(dev.freed_count.item())
    assert torch.equal(dev.freed[:nf], host.freed[:nf])
    assert torch.equal(dev.layers[0].k_pool, host.layers[0].k_pool)
    # and the oracle, once more, through the device-planned step
    want, _ = oracle_attn(A)
    mx, mean, rel = attn_errors(dev.out[0][:tq], want)
    assert mx <= 2e-2 and mean <= 2e-3 and rel <= 1e-2, (mx, mean, rel)
    acc = oracle_accept(A)
    assert np.array_equal(dev.accept_len.cpu().numpy()[:B], acc["accept_len"])


def test_device_plan_takes_pages_from_a_device_free_list(bnd):
    """Pages for the draft positions come from a free list in device memory: same table as the host planner writes."""
    A = _batch(11, 128, 16, 4, 0, 6, 5)
    held = (A.seq_lens.astype(np.int64) + A.block_size - 1) // A.block_size
    need = (A.seq_lens.astype(np.int64) + A.draft_lens + 1 + A.block_size - 1) // A.block_size
    table = A.block_table.copy()
    free = []
    for i in range(A.batch):                               # hand the draft pages back, in (request, page) order
        free += list(table[i, held[i]:need[i]])
        table[i, held[i]:need[i]] = -1
    free = np.asarray(free + [0] * 3, dtype=np.int32)      # a few entries more than needed
    B = copy.copy(A)
    B.block_table = table
    host, dev = bnd.VerifyStep(B), bnd.VerifyStep(B)
    for s in (host, dev):
        bnd.as_plan_set_fixed_launch(s.plan, True)
    taken = bnd.as_plan(host.plan, B.seq_lens, B.draft_lens, host.block_table, free_blocks=free)
    assert taken == int((need - held).sum())
    bnd.as_plan_device(dev.plan, B.batch, dev.seq_lens, torch.as_tensor(B.draft_lens, dtype=torch.int32, device="cuda"),
                       dev.block_table, torch.as_tensor(free, device="cuda"), len(free))
    host.attn(0); dev.attn(0)
    torch.cuda.synchronize()
    assert bnd.as_plan_check(dev.plan) == 0
    assert torch.equal(dev.block_table, host.block_table)
    assert np.array_equal(dev.block_table.cpu().numpy(), A.block_table)
    assert torch.equal(dev.out[0][:A.total_q], host.out[0][:A.total_q])


@pytest.mark.parametrize("what", ["draft_len", "seq_len", "pages", "free_list"])
def test_device_plan_rejects_bad_lengths_with_a_flag_and_an_empty_step(bnd, what):
    A = _batch(21, 128, 8, 2, 0, 4, 3)
    vs = bnd.VerifyStep(A)
    bnd.as_plan_set_fixed_launch(vs.plan, True)
    seq = torch.as_tensor(A.seq_lens, dtype=torch.int32, device="cuda")
    dl = torch.as_tensor(A.draft_lens, dtype=torch.int32, device="cuda")
    free, num_free = None, 0
    if what == "draft_len":
        dl[1] = A.k_max + 1
    elif what == "seq_len":
        seq[2] = -5
    elif what == "pages":
        seq[0] = A.max_blocks * A.block_size             # needs one page more than a table row holds
    else:
        free, num_free = torch.zeros(1, dtype=torch.int32, device="cuda"), 1   # every request needs at least one new page
        seq = seq // A.block_size * A.block_size          # (so that position n is the first of a fresh page)
    vs.seq_lens.copy_(seq)
    before = [t.clone() for t in (vs.out[0], vs.accept_len, vs.seq_lens, vs.block_table, vs.layers[0].k_pool)]
    bnd.as_plan_device(vs.plan, A.batch, vs.seq_lens, dl, vs.block_table, free, num_free)
    vs.attn(0); vs.accept(); vs.commit()
    torch.cuda.synchronize()
    assert bnd.as_plan_check(vs.plan, raise_on_flag=False) & bnd.AS_FLAG_BAD_PLAN
    after = (vs.out[0], vs.accept_len, vs.seq_lens, vs.block_table, vs.layers[0].k_pool)
    assert all(torch.equal(x, y) for x, y in zip(before, after))
    # the plan is usable again at once
    vs.seq_lens.copy_(torch.as_tensor(A.seq_lens, device="cuda"))
    bnd.as_plan_device(vs.plan, A.batch, vs.seq_lens, torch.as_tensor(A.draft_lens, dtype=torch.int32, device="cuda"), vs.block_table)
    vs.attn(0)
    torch.cuda.synchronize()
    assert bnd.as_plan_check(vs.plan) == 0
    want, _ = oracle_attn(A)
    mx, mean, rel = attn_errors(vs.out[0][:A.total_q], want)
    assert mx <= 2e-2 and mean <= 2e-3


def _free_ids(block_table: torch.Tensor, num_blocks: int, size: int) -> np.ndarray:
    used = set(int(x) for x in block_table.cpu().numpy().ravel() if x >= 0)
    free = [i for i in range(num_blocks) if i not in used]
    assert len(free) >= 1
    return np.asarray((free + [free[0]] * size)[:size], dtype=np.int32)   # padded; the padding is never reached


def test_recorded_step_with_device_plan_replays_while_lengths_evolve_on_the_device(bnd):
    """plan + attention + acceptance + commit recorded once; four replays, each starting from the seq_lens and the
    block table the previous commit left on the device; a host-planned twin does the same steps with ordinary launches."""
    B, kmax = 5, 4
    A = workloads.make_batch("pd_multi", seed=31, seq_lens=[300, 17, 1000, 0, 129], draft_lens=[kmax] * B, num_q_heads=16,
                             num_kv_heads=4, head_dim=128, vocab=400, logit_std=2.0, match="iid", match_p=0.7, k_max=kmax)
    dev, ref = bnd.VerifyStep(A), bnd.VerifyStep(A)
    bnd.as_plan_set_fixed_launch(dev.plan, True)
    nfree = 4 * B
    free_dev = torch.zeros(nfree, dtype=torch.int32, device="cuda")
    dl_dev = torch.zeros(B, dtype=torch.int32, device="cuda")

    def one_step(draft_lens):
        dl_dev.copy_(torch.as_tensor(draft_lens, dtype=torch.int32))
        free = _free_ids(dev.block_table, A.num_blocks, nfree)
        free_dev.copy_(torch.as_tensor(free))
        return free

    def record():
        bnd.as_plan_device(dev.plan, B, dev.seq_lens, dl_dev, dev.block_table, free_dev, nfree)
        dev.attn(0); dev.accept(); dev.commit()

    # the draft pages of the first step go back to the free list, so that every step takes its pages the same way
    for s in (dev, ref):
        held = (A.seq_lens.astype(np.int64) + A.block_size - 1) // A.block_size
        bt = s.block_table.cpu().numpy()
        for i in range(B):
            bt[i, held[i]:] = -1
        s.block_table.copy_(torch.as_tensor(bt))
    one_step([kmax] * B)
    bt0, seq0 = dev.block_table.clone(), dev.seq_lens.clone()
    record()                                               # once unrecorded
    torch.cuda.synchronize()
    dev.block_table.copy_(bt0); dev.seq_lens.copy_(seq0)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        record()
    torch.cuda.synchronize()
    dev.block_table.copy_(bt0); dev.seq_lens.copy_(seq0)

    for step, draft_lens in enumerate([[4, 4, 4, 4, 4], [0, 3, 4, 1, 2], [2, 2, 0, 4, 4], [4, 0, 1, 3, 0]]):
        free = one_step(draft_lens)
        seq_now = ref.seq_lens.cpu().numpy()
        assert np.array_equal(seq_now, dev.seq_lens.cpu().numpy())
        graph.replay()
        V = copy.copy(A)
        V.seq_lens, V.draft_lens = seq_now.astype(np.int32), np.asarray(draft_lens, dtype=np.int32)
        ref.set_batch(V)
        bnd.as_plan(ref.plan, V.seq_lens, V.draft_lens, ref.block_table, free_blocks=free)
        ref.attn(0); ref.accept(); ref.commit()
        torch.cuda.synchronize()
        assert bnd.as_plan_check(dev.plan) == 0 and bnd.as_plan_check(ref.plan) == 0, step
        tq = int(np.sum(draft_lens)) + B
        assert torch.equal(dev.out[0][:tq], ref.out[0][:tq]), step
        assert torch.equal(dev.accept_len[:B], ref.accept_len[:B]) and torch.equal(dev.out_tokens[:B], ref.out_tokens[:B]), step
        assert torch.equal(dev.seq_lens, ref.seq_lens) and torch.equal(dev.block_table, ref.block_table), step
        assert torch.equal(dev.layers[0].k_pool, ref.layers[0].k_pool), step
    assert int(dev.seq_lens.sum().item()) > int(seq0.sum().item())          # the contexts did grow


def test_two_layer_kinds_planned_on_the_device(bnd):
    """A windowed and a full layer (head_dim 64, the rows-on-M kernel, sinks): both work lists come from one plan_kernel."""
    g = torch.Generator().manual_seed(3)
    kinds = [workloads.LayerKind(window=128, sinks=torch.randn(64, generator=g)),
             workloads.LayerKind(window=0, sinks=torch.randn(64, generator=g))]
    A = workloads.make_batch("pd2", seed=41, seq_lens=[5000, 300, 127, 20000, 64], draft_lens=[16, 3, 0, 9, 12], num_q_heads=64,
                             num_kv_heads=8, head_dim=64, vocab=300, logit_std=2.0, match="markov", k_max=16, kinds=kinds)
    host, dev = bnd.VerifyStep(A), bnd.VerifyStep(A)
    for s in (host, dev):
        bnd.as_plan_set_fixed_launch(s.plan, True)
    host.plan_step()
    dev.plan_step_device(A.batch, torch.as_tensor(A.draft_lens, dtype=torch.int32, device="cuda"))
    for kind in (0, 1):
        host.attn(kind); dev.attn(kind)
    host.accept(); dev.accept(); host.commit(kind=1); dev.commit(kind=1)
    torch.cuda.synchronize()
    assert bnd.as_plan_check(host.plan) == 0 and bnd.as_plan_check(dev.plan) == 0
    tq = A.total_q
    for kind in (0, 1):
        assert torch.equal(dev.out[kind][:tq], host.out[kind][:tq]) and torch.equal(dev.lse[kind][:tq], host.lse[kind][:tq])
        want, _ = oracle_attn(A, kind=kind)
        mx, mean, rel = attn_errors(dev.out[kind][:tq], want)
        assert mx <= 2e-2 and mean <= 2e-3 and rel <= 1e-2, (kind, mx, mean, rel)
    assert torch.equal(dev.accept_len, host.accept_len) and torch.equal(dev.seq_lens, host.seq_lens)
    assert torch.equal(dev.block_table, host.block_table)


def test_argument_checks_of_the_new_entry_points(bnd):
    A = _batch(51, 128, 8, 2, 0, 3, 2)
    vs = bnd.VerifyStep(A)
    dl = torch.as_tensor(A.draft_lens, dtype=torch.int32, device="cuda")
    with pytest.raises(bnd.AsError):                       # the device planner needs fixed launches
        bnd.as_plan_device(vs.plan, A.batch, vs.seq_lens, dl, vs.block_table)
    bnd.as_plan_set_fixed_launch(vs.plan, True)
    with pytest.raises(bnd.AsError):
        bnd.as_plan_device(vs.plan, A.batch + 1, vs.seq_lens, dl, vs.block_table)      # more requests than the plan holds
    hidden = torch.zeros((A.batch * (A.k_max + 1), 96), dtype=torch.bfloat16, device="cuda")
    weight = torch.zeros((A.vocab, 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bnd.AsError):                       # no plan for this step yet
        bnd.as_accept_lm_head(vs.plan, hidden, weight, vs.draft_tokens, vs.accept_len, vs.out_tokens)
    bnd.as_plan_device(vs.plan, A.batch, vs.seq_lens, dl, vs.block_table)
    with pytest.raises(bnd.AsError):                       # hidden size must be a multiple of 64
        bnd.as_accept_lm_head(vs.plan, hidden, weight, vs.draft_tokens, vs.accept_len, vs.out_tokens)
    torch.cuda.synchronize()
    assert bnd.as_plan_check(vs.plan) == 0
