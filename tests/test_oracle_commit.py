"""Pins for the oracle's KV commit / rollback, and the whole-step losslessness loop."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_24004_b200 import workloads
from helpers import np_bits, oracle_attn, oracle_commit, gather_logical, cu


def _hand_batch():
    # page size 4, n = 6 cached, k = 5 drafts: positions 6..11 are tentative, pages 0..2 are held
    return workloads.make_batch("t", seed=1, seq_lens=[6], draft_lens=[5], num_q_heads=2, num_kv_heads=1, head_dim=4,
                                vocab=8, block_size=4, with_logits=False)


@pytest.mark.parametrize("a,n_new,freed_logical", [(0, 7, [2]), (1, 8, [2]), (2, 9, []), (5, 12, [])])
def test_hand_worked_paging(a, n_new, freed_logical):
    """n' = n + a + 1.  a = 0 -> 7 entries: pages 0-1 kept, page 2 released.  a = 1 -> 8 entries fill
    page 1 exactly, page 2 released.  a = 2 -> 9 entries reach into page 2, kept.  a = 5 -> all kept."""
    b = _hand_batch()
    before = b.block_table.copy()
    seq, bt, kp, vp, freed = oracle_commit(b, [a])
    assert list(seq) == [n_new]
    assert list(freed) == [int(before[0, l]) for l in freed_logical]
    keep = math.ceil(n_new / 4)
    assert (bt[0, keep:] == -1).all() and (bt[0, :keep] == before[0, :keep]).all()
    # logical contents: the old 6 entries followed by the first a+1 staging rows, bit for bit
    L = b.layers[0]
    got_k = gather_logical(kp, bt[0], n_new, 4)
    want_k = np.concatenate([gather_logical(np_bits(L.k_pool), before[0], 6, 4), np_bits(L.k_new)[:a + 1]])
    assert np.array_equal(got_k, want_k)
    got_v = gather_logical(vp, bt[0], n_new, 4)
    want_v = np.concatenate([gather_logical(np_bits(L.v_pool), before[0], 6, 4), np_bits(L.v_new)[:a + 1]])
    assert np.array_equal(got_v, want_v)


@pytest.mark.parametrize("a,freed_logical", [(0, [2]), (2, []), (5, [])])
def test_table_entries_past_the_steps_pages_are_not_released(a, freed_logical):
    """Which pages a rollback releases: only those the STEP held, i.e. logical pages in
    [ceil(n'/bs), ceil((n+k+1)/bs)).  A scheduler may have reserved pages further out in the same block-table row
    (here logical pages 3 and 4, beyond the step's last position 11): they are not the step's to give back, so they
    stay in the table and never show up in the freed list, whatever is accepted."""
    b = _hand_batch()
    assert b.block_table.shape[1] >= 5 and (b.block_table[0, 3:5] == -1).all()
    spare = [p for p in range(64) if p not in set(b.block_table[0, :3].tolist())][:2]
    b.block_table[0, 3:5] = spare
    before = b.block_table.copy()
    seq, bt, kp, vp, freed = oracle_commit(b, [a])
    assert list(seq) == [6 + a + 1]
    assert list(freed) == [int(before[0, l]) for l in freed_logical]
    assert list(bt[0, 3:5]) == spare
    keep = math.ceil((6 + a + 1) / 4)
    assert (bt[0, keep:3] == -1).all() and (bt[0, :keep] == before[0, :keep]).all()


def test_scrub_zeroes_rejected_slots_in_held_pages_only():
    b = _hand_batch()
    seq, bt, kp, vp, freed = oracle_commit(b, [2], scrub=True)        # n' = 9: slot 0 of page 2 kept
    page2 = bt[0, 2]
    assert (kp[page2, :, 1:] == 0).all() and (vp[page2, :, 1:] == 0).all()
    assert (kp[page2, :, 0] != 0).any()
    # other pages untouched
    for l in (0, 1):
        assert np.array_equal(kp[bt[0, l]], np.where(True, kp[bt[0, l]], 0))
    _, _, kp2, _, _ = oracle_commit(b, [2], scrub=False)
    assert np.array_equal(kp2[page2, :, 0], kp[page2, :, 0])


def test_multi_request_freed_order_and_poison():
    b = workloads.make_batch("t", seed=2, seq_lens=[14, 3, 31], draft_lens=[6, 0, 8], num_q_heads=2, num_kv_heads=1,
                             head_dim=4, vocab=8, block_size=4, with_logits=False)
    before = b.block_table.copy()
    seq, bt, kp, vp, freed = oracle_commit(b, [0, 0, 1])
    # request 0: n' = 15 -> keep 4 pages of 6 held (ceil(21/4)); request 1: nothing; request 2: n' = 33 -> keep 9 of 10
    assert list(seq) == [15, 4, 33]
    assert list(freed) == [before[0, 4], before[0, 5], before[2, 9]]
    # poison: whatever sits in rejected slots of still-held pages cannot influence the next k=0 step
    nxt = workloads.make_batch("t", seed=3, seq_lens=seq, draft_lens=[0, 0, 0], num_q_heads=2, num_kv_heads=1,
                               head_dim=4, vocab=8, block_size=4, with_logits=False)
    nb = max(nxt.num_blocks, b.num_blocks)
    def run(kpool, vpool):
        return oracle.verify_attn(seq, [0, 0, 0], np_bits(nxt.layers[0].q), np_bits(nxt.layers[0].k_new),
                                  np_bits(nxt.layers[0].v_new), kpool, vpool, np.where(bt < 0, 0, bt),
                                  num_q_heads=2, num_kv_heads=1, head_dim=4, block_size=4)[0]
    ref = run(kp, vp)
    kp2, vp2 = kp.copy(), vp.copy()
    for i in range(3):
        for t in range(int(seq[i]), (int(seq[i]) + 3) // 4 * 4):
            kp2[bt[i, t // 4], :, t % 4] = 0x7F80   # +inf
            vp2[bt[i, t // 4], :, t % 4] = 0x7FC0   # NaN
    assert np.array_equal(run(kp2, vp2), ref)


# ---------------------------------------------------------------- greedy speculation == autoregression

class ToyModel:
    """Deterministic one-layer 'model': Q/K/V of a token at a position come from fixed random
    bf16 tables, the logits are a fixed fp64 read-out of the attention output."""

    def __init__(self, seed=0, V=48, Hq=4, Hkv=2, D=8):
        g = torch.Generator().manual_seed(seed)
        self.V, self.Hq, self.Hkv, self.D = V, Hq, Hkv, D
        self.Eq = torch.randn(V, Hq, D, generator=g); self.Pq = torch.randn(16, Hq, D, generator=g)
        self.Ek = torch.randn(V, Hkv, D, generator=g); self.Pk = torch.randn(16, Hkv, D, generator=g)
        self.Ev = torch.randn(V, Hkv, D, generator=g)
        self.W = torch.randn(V, Hq * D, generator=g, dtype=torch.float64).numpy()

    def qkv(self, tokens, positions):
        t = torch.as_tensor(tokens, dtype=torch.long); p = torch.as_tensor(positions, dtype=torch.long) % 16
        return ((self.Eq[t] + self.Pq[p]).bfloat16(), (self.Ek[t] + self.Pk[p]).bfloat16(), self.Ev[t].bfloat16())

    def logits(self, attn_out):          # [rows, Hq, D] fp64 -> [rows, V] fp32
        return (attn_out.reshape(len(attn_out), -1) @ self.W.T).astype(np.float32)


def _step(model, seqs, n, ks, drafts, bt, kpool, vpool, bs):
    """One verify step through the oracle: attention -> logits -> greedy accept -> commit."""
    toks, pos = [], []
    for i in range(len(seqs)):
        toks += [seqs[i][n[i]]] + list(drafts[i]); pos += list(range(n[i], n[i] + ks[i] + 1))
    q, kn, vn = model.qkv(toks, pos)
    out, _ = oracle.verify_attn(n, ks, np_bits(q), np_bits(kn), np_bits(vn), kpool, vpool, np.where(bt < 0, 0, bt),
                                num_q_heads=model.Hq, num_kv_heads=model.Hkv, head_dim=model.D, block_size=bs)
    z = model.logits(out)
    flat = [d for dr in drafts for d in dr]
    acc = oracle.accept(ks, z, model.V, flat, k_max=max(max(ks), 1))
    seq2, bt2, kp2, vp2, freed = oracle.kv_commit(n, ks, acc["accept_len"], bt, np_bits(kn), np_bits(vn), kpool, vpool,
                                                  num_kv_heads=model.Hkv, head_dim=model.D, block_size=bs)
    return acc, seq2, bt2, kp2, vp2, freed


def test_greedy_speculative_loop_equals_autoregressive_loop():
    model = ToyModel()
    bs, T, B = 4, 60, 2
    rng = np.random.default_rng(5)
    prompts = [list(rng.integers(0, model.V, size=5)), list(rng.integers(0, model.V, size=9))]
    max_blocks = 40
    num_blocks = B * max_blocks

    def fresh_state():
        free = list(rng.permutation(num_blocks))
        bt = np.full((B, max_blocks), -1, np.int32)
        kpool = np.zeros((num_blocks, model.Hkv, bs, model.D), np.uint16); vpool = kpool.copy()
        n = []
        for i, pr in enumerate(prompts):         # prefill all but the last prompt token
            _, k, v = model.qkv(pr[:-1], list(range(len(pr) - 1)))
            for t in range(len(pr) - 1):
                if bt[i, t // bs] < 0:
                    bt[i, t // bs] = free.pop()
                kpool[bt[i, t // bs], :, t % bs] = np_bits(k[t]); vpool[bt[i, t // bs], :, t % bs] = np_bits(v[t])
            n.append(len(pr) - 1)
        return free, bt, kpool, vpool, n

    def ensure_pages(free, bt, n, ks):
        for i in range(B):
            for l in range((n[i] + ks[i] + 1 + bs - 1) // bs):
                if bt[i, l] < 0:
                    bt[i, l] = free.pop()

    # autoregressive: k = 0 every step
    free, bt, kpool, vpool, n = fresh_state()
    seqs = [list(p) for p in prompts]
    for _ in range(T):
        ensure_pages(free, bt, n, [0] * B)
        acc, n2, bt, kpool, vpool, freed = _step(model, seqs, n, [0] * B, [[] for _ in range(B)], bt, kpool, vpool, bs)
        assert len(freed) == 0 and list(acc["accept_len"]) == [0] * B
        for i in range(B):
            seqs[i].append(int(acc["out_tokens"][i, 0]))
        n = [int(x) for x in n2]
    ar_seqs = seqs
    ar_cache = [(gather_logical(kpool, bt[i], n[i], bs), gather_logical(vpool, bt[i], n[i], bs)) for i in range(B)]

    # speculative: drafts = the true continuation with random corruptions, random k in 0..6
    free, bt, kpool, vpool, n = fresh_state()
    seqs = [list(p) for p in prompts]
    steps = 0
    total_acc = 0
    while min(len(s) for s in seqs) < min(len(s) for s in ar_seqs):
        ks, drafts = [], []
        for i in range(B):
            room = len(ar_seqs[i]) - len(seqs[i]) - 1
            k = int(min(rng.integers(0, 7), max(room, 0)))
            d = list(ar_seqs[i][len(seqs[i]):len(seqs[i]) + k])
            for j in range(k):
                if rng.random() < 0.25:
                    d[j] = int((d[j] + 1 + rng.integers(0, model.V - 1)) % model.V)
            ks.append(k); drafts.append(d)
        ensure_pages(free, bt, n, ks)
        acc, n2, bt, kpool, vpool, freed = _step(model, seqs, n, ks, drafts, bt, kpool, vpool, bs)
        free += [int(x) for x in freed]
        for i in range(B):
            a = int(acc["accept_len"][i])
            new = [int(x) for x in acc["out_tokens"][i, :a + 1]]
            seqs[i] += new                                     # a finished request just keeps decoding
            total_acc += a
        n = [int(x) for x in n2]
        steps += 1
        assert steps < 10 * T
    assert total_acc > 20                                      # speculation did accept tokens
    for i in range(B):
        m = min(len(seqs[i]), len(ar_seqs[i]))
        assert seqs[i][:m] == ar_seqs[i][:m]                   # token-for-token the same text
        c = min(n[i], len(ar_cache[i][0]))
        assert np.array_equal(gather_logical(kpool, bt[i], c, bs), ar_cache[i][0][:c])     # same cache, bit for bit
        assert np.array_equal(gather_logical(vpool, bt[i], c, bs), ar_cache[i][1][:c])
        held = int((bt[i] >= 0).sum())
        assert held == (n[i] + bs - 1) // bs                   # no leaked pages
    assert len(free) + int((bt >= 0).sum()) == num_blocks and len(set(free)) == len(free)
