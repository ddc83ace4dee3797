"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs.

Tolerances (written where they are applied): KV commit / rollback and greedy acceptance are
bit-exact; attention output max-abs <= 2e-2 and mean-abs <= 2e-3 (plus, because those absolute bounds
are about the size of the signal at long context, relative Frobenius error <= 1e-2 and
|lse - lse*| <= 1e-3); sampled accept decisions exact except where the oracle's min(1, p/q) lies within
1e-5 of the uniform (those positions are counted and must stay under 1e-4 of positions).
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_24004_b200 import workloads
from helpers import np_bits, oracle_attn, oracle_accept, oracle_commit, gather_logical, cu, attn_errors

pytestmark = pytest.mark.gpu

ATTN_MAX_ABS, ATTN_MEAN_ABS, ATTN_REL_FRO, LSE_ABS = 2e-2, 2e-3, 1e-2, 1e-3


@pytest.fixture(scope="module")
def bnd():
    from paper_2608_24004_b200 import build as as_build
    as_build.build_library()
    from paper_2608_24004_b200 import binding
    return binding


def impls(bnd):
    return [bnd.AS_ATTN_SIMT, bnd.AS_ATTN_TC]


def run_attn(bnd, batch, impl, kind=0):
    """Plans and runs one attention layer; returns (VerifyStep, out bf16, lse fp32) or None if the
    forced kernel does not cover the shape."""
    vs = bnd.VerifyStep(batch, attn_impl=impl)
    try:
        vs.plan_step()
    except bnd.AsError as e:
        if e.status == bnd.AS_ERR_UNSUPPORTED and impl == bnd.AS_ATTN_TC:
            return None
        raise
    vs.attn(kind)
    assert bnd.as_plan_check(vs.plan) == 0
    return vs, vs.out[kind], vs.lse[kind]


def check_attn(out, lse, want, want_lse, exact_rows=None):
    mx, mean, rel = attn_errors(out, want)
    assert mx <= ATTN_MAX_ABS and mean <= ATTN_MEAN_ABS and rel <= ATTN_REL_FRO, (mx, mean, rel)
    assert np.abs(lse.double().cpu().numpy() - want_lse).max() <= LSE_ABS


@pytest.mark.parametrize("impl_i", [0, 1])
def test_tiny_config_whole_step(bnd, impl_i):
    impl = impls(bnd)[impl_i]
    b = workloads.tiny()
    want, want_lse = oracle_attn(b)
    r = run_attn(bnd, b, impl)
    if r is None:
        pytest.skip("tensor-core kernel does not cover this shape")
    vs, out, lse = r
    check_attn(out, lse, want, want_lse)
    # greedy acceptance: bit exact
    vs.accept()
    acc = oracle_accept(b)
    assert np.array_equal(vs.accept_len.cpu().numpy(), acc["accept_len"])
    assert np.array_equal(vs.out_tokens.cpu().numpy(), acc["out_tokens"])
    # commit: the pools now hold the appended rows; compare the observable state
    vs.commit(flags=bnd.AS_COMMIT_SCRUB)
    assert bnd.as_plan_check(vs.plan) == 0
    seq, bt, kp, vp, freed = oracle_commit(b, acc["accept_len"], scrub=True)
    assert np.array_equal(vs.seq_lens.cpu().numpy(), seq)
    assert np.array_equal(vs.block_table.cpu().numpy(), bt)
    nf = int(vs.freed_count.item())
    assert np.array_equal(vs.freed.cpu().numpy()[:nf], freed)
    gk, gv = np_bits(vs.layers[0].k_pool), np_bits(vs.layers[0].v_pool)
    for i in range(b.batch):
        keep_to = -(-int(seq[i]) // b.block_size) * b.block_size          # scrubbed up to the end of the last held page
        upto = min(keep_to, int(b.seq_lens[i] + b.draft_lens[i] + 1))
        assert np.array_equal(gather_logical(gk, bt[i], upto, b.block_size), gather_logical(kp, bt[i], upto, b.block_size))
        assert np.array_equal(gather_logical(gv, bt[i], upto, b.block_size), gather_logical(vp, bt[i], upto, b.block_size))


SHAPES = [
    # (Hq, Hkv, D, bs, window, sinks, seq_lens, draft_lens)
    (8, 2, 128, 16, 0, False, [0, 1, 15, 16, 17, 300], [0, 3, 4, 0, 8, 2]),
    (32, 8, 128, 16, 0, False, [700, 129, 2100], [8, 0, 5]),
    (32, 8, 128, 32, 0, True, [513, 127, 128], [1, 7, 4]),
    (64, 8, 64, 16, 0, True, [1000, 50], [16, 3]),
    (64, 8, 64, 16, 128, True, [1000, 50, 127, 128, 129, 400], [16, 3, 0, 5, 9, 12]),
    (8, 8, 64, 64, 40, False, [333, 20], [4, 6]),
    (4, 1, 128, 128, 0, False, [260, 4000], [2, 2]),
    (16, 4, 128, 16, 200, False, [5000, 190, 201], [6, 6, 6]),
    (32, 8, 128, 16, 0, False, [900, 33, 1], [23, 15, 19]),          # 96, 64 and 80 rows: the widest head_dim-128 tiles
    (64, 8, 64, 16, 0, True, [700, 260, 5], [11, 5, 7]),             # 96, 48 and 64 rows at head_dim 64
    (32, 8, 128, 16, 0, True, [2500, 140, 260], [27, 24, 25]),       # 112, 100 and 104 rows: seven softmax warpgroups
    (64, 8, 128, 32, 0, False, [700, 129], [13, 12]),                # 112 and 104 rows with eight query heads per kv head
    (64, 8, 128, 16, 0, True, [1500, 129, 40], [15, 14, 15]),        # 128 and 120 rows: eight slabs on seven warpgroups
    (64, 8, 64, 16, 0, False, [300, 5000, 127], [17, 15, 16]),       # 144, 128 and 136 rows: one and two blocks of 128 rows
    (64, 8, 64, 32, 300, True, [40000, 299, 300, 301], [16, 17, 0, 9]),   # two row blocks under a window, one long split pair
    (8, 8, 64, 16, 0, False, [1000, 129, 0], [16, 1, 0]),            # one query head per kv head: 17, 2 and 1 rows
    (64, 8, 64, 16, 0, True, [500, 3000, 64], [31, 20, 24]),         # 256, 168 and 200 rows: the most head_dim 64 takes
    (64, 8, 128, 16, 0, True, [1500, 129, 40, 5000], [16, 15, 16, 0]),   # head_dim 128 beyond 128 rows: 136 = two row blocks
    (64, 8, 128, 16, 0, False, [700, 2600, 127], [23, 17, 31]),      # 192, 144 and 256 rows at head_dim 128
    (64, 8, 128, 32, 200, True, [40000, 199, 200, 201], [31, 16, 24, 5]),   # row blocks under a window, one long split pair
    (48, 16, 128, 16, 0, False, [900, 300], [60, 41]),               # three query heads per kv head: blocks of 42 positions
    (16, 2, 64, 128, 0, False, [260, 4000, 130], [2, 9, 0]),         # head_dim 64 with one page per tile
]


@pytest.mark.parametrize("impl_i", [0, 1])
@pytest.mark.parametrize("shape_i", range(len(SHAPES)))
def test_attention_shapes(bnd, shape_i, impl_i):
    Hq, Hkv, D, bs, window, sinks, seq, dl = SHAPES[shape_i]
    g = torch.Generator().manual_seed(shape_i)
    kinds = [workloads.LayerKind(window=window, sinks=torch.randn(Hq, generator=g) if sinks else None)]
    b = workloads.make_batch("t", seed=100 + shape_i, seq_lens=seq, draft_lens=dl, num_q_heads=Hq, num_kv_heads=Hkv,
                             head_dim=D, vocab=8, block_size=bs, kinds=kinds, with_logits=False)
    r = run_attn(bnd, b, impls(bnd)[impl_i])
    if r is None:
        pytest.skip("tensor-core kernel does not cover this shape")
    _, out, lse = r
    want, want_lse = oracle_attn(b)
    check_attn(out, lse, want, want_lse)


@pytest.mark.parametrize("impl_i", [0, 1])
@pytest.mark.parametrize("D,draft_lens", [(128, [0, 2, 1]), (64, [3, 0, 0]), (64, [0, 0, 0])])
def test_plan_capacity_larger_than_the_steps_drafts(bnd, impl_i, D, draft_lens):
    """A plan created for 16 drafts per request serving a step whose longest draft is short: the kernel
    instance follows the step, not the plan's capacity, and the results do not change."""
    b = workloads.make_batch("t", seed=41, seq_lens=[700, 129, 2500], draft_lens=draft_lens, num_q_heads=32 if D == 128 else 64,
                             num_kv_heads=8, head_dim=D, vocab=8, with_logits=False, k_max=16)
    r = run_attn(bnd, b, impls(bnd)[impl_i])
    if r is None:
        pytest.skip("tensor-core kernel does not cover this shape")
    _, out, lse = r
    want, want_lse = oracle_attn(b)
    check_attn(out, lse, want, want_lse)


def _random_shape(seed):
    """A random small configuration inside what the library accepts: head layout, head_dim, page size,
    window, sinks, a ragged mix of context lengths (page and tile boundaries included) and draft lengths."""
    rng = np.random.default_rng(1000 + seed)
    D = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 8]))
    bs = int(rng.choice([16, 32, 64, 128]))
    max_rows = 256 if D == 64 else 128
    kmax = int(rng.integers(0, min(31, max_rows // G - 1) + 1))
    window = int(rng.choice([0, 0, int(rng.integers(1, 400))]))
    B = int(rng.integers(1, 7))
    edges = np.array([0, 1, bs - 1, bs, bs + 1, 127, 128, 129, 255, 256, 257])
    seq = [int(rng.choice(edges)) if rng.random() < 0.4 else int(rng.integers(0, 3000)) for _ in range(B)]
    dl = [int(rng.integers(0, kmax + 1)) for _ in range(B)]
    dl[int(rng.integers(0, B))] = kmax
    return G * Hkv, Hkv, D, bs, window, bool(rng.random() < 0.5), seq, dl


@pytest.mark.parametrize("impl_i", [0, 1])
@pytest.mark.parametrize("seed", range(24))
def test_attention_random_shapes(bnd, seed, impl_i):
    Hq, Hkv, D, bs, window, sinks, seq, dl = _random_shape(seed)
    g = torch.Generator().manual_seed(seed)
    kinds = [workloads.LayerKind(window=window, sinks=torch.randn(Hq, generator=g) if sinks else None)]
    b = workloads.make_batch("t", seed=500 + seed, seq_lens=seq, draft_lens=dl, num_q_heads=Hq, num_kv_heads=Hkv,
                             head_dim=D, vocab=8, block_size=bs, kinds=kinds, with_logits=False)
    r = run_attn(bnd, b, impls(bnd)[impl_i])
    if r is None:
        pytest.skip("tensor-core kernel does not cover this shape")
    _, out, lse = r
    want, want_lse = oracle_attn(b)
    check_attn(out, lse, want, want_lse)


@pytest.mark.parametrize("impl_i", [0, 1])
@pytest.mark.parametrize("window,sink", [(0, None), (0, 0.5), (128, None), (37, -1.0)])
def test_uniform_softmax_counts_visible_keys(bnd, impl_i, window, sink):
    """K = 0: every score is 0 and the output is a plain mean over the visible range, so a dropped
    page, an off-by-one causal edge or a wrong window edge changes out[1] by O(1/c).  All inputs are
    bf16-exact; the only error is the bf16 rounding of the output."""
    n, k, bs, D, Hq, Hkv = [1300, 77, 16, 2047, 129], [3, 0, 8, 5, 8], 16, 128, 8, 2
    b = workloads.make_batch("t", seed=3, seq_lens=n, draft_lens=k, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D,
                             vocab=8, block_size=bs, with_logits=False,
                             kinds=[workloads.LayerKind(window=window,
                                                        sinks=None if sink is None else torch.full((Hq,), sink))])
    L = b.layers[0]
    L.k_pool.zero_(); L.k_new.zero_(); L.v_pool.zero_(); L.v_new.zero_()
    cu_q, _ = cu(b.draft_lens)
    for i in range(len(n)):
        t = torch.arange(n[i] + k[i] + 1)
        val = torch.zeros(len(t), Hkv, D, dtype=torch.bfloat16)
        val[:, :, 0] = 1.0
        val[:, :, 1] = (t % 64).to(torch.bfloat16)[:, None]
        blocks = torch.as_tensor(b.block_table[i, (t[:n[i]] // bs).numpy()], dtype=torch.long)
        L.v_pool[blocks, :, t[:n[i]] % bs] = val[:n[i]]
        L.v_new[cu_q[i]:cu_q[i + 1]] = val[n[i]:]
    r = run_attn(bnd, b, impls(bnd)[impl_i])
    if r is None:
        pytest.skip("tensor-core kernel does not cover this shape")
    _, out, lse = r
    out = out.float().cpu().numpy(); lse = lse.cpu().numpy()
    for i in range(len(n)):
        for j in range(k[i] + 1):
            p = n[i] + j
            lo = max(0, p - window + 1) if window > 0 else 0
            c = p - lo + 1
            es = 0.0 if sink is None else math.exp(sink)
            w0 = c / (c + es)
            w1 = sum(t % 64 for t in range(lo, p + 1)) / (c + es)
            row = out[cu_q[i] + j]
            assert np.abs(row[:, 0] - w0).max() <= 2 ** -8 * w0 + 1e-6, (i, j)
            assert np.abs(row[:, 1] - w1).max() <= 2 ** -7 * w1 + 1e-3, (i, j)        # bf16 weights and output
            assert np.abs(lse[cu_q[i] + j] - math.log(c + es)).max() <= 1e-4, (i, j)


@pytest.mark.parametrize("impl_i", [0, 1])
def test_needle_positions(bnd, impl_i):
    """One dominant key per run (q.k = 40 sqrt(D)): the output must be that key's value to bf16.
    Positions: first / last of the context, page edges, tile edges, every new row."""
    n, k, bs, D = 700, 4, 16, 128
    b = workloads.make_batch("t", seed=5, seq_lens=[n], draft_lens=[k], num_q_heads=4, num_kv_heads=1, head_dim=D,
                             vocab=8, block_size=bs, with_logits=False)
    L = b.layers[0]
    L.k_pool.zero_(); L.k_new.zero_()
    L.q.zero_(); L.q[:, :, 0] = 1.0
    vs = None
    for t in [0, 1, 15, 16, 17, 127, 128, 129, 255, 256, 511, 512, 639, 640, 698, 699, 700, 701, 702, 703, 704]:
        kp, kn = L.k_pool.clone(), L.k_new.clone()
        if t < n:
            L.k_pool[b.block_table[0, t // bs], 0, t % bs, 0] = 40.0 * math.sqrt(D)
            want = L.v_pool[b.block_table[0, t // bs], 0, t % bs]
        else:
            L.k_new[t - n, 0, 0] = 40.0 * math.sqrt(D)
            want = L.v_new[t - n, 0]
        r = run_attn(bnd, b, impls(bnd)[impl_i])
        if r is None:
            pytest.skip("tensor-core kernel does not cover this shape")
        _, out, _ = r
        for j in range(k + 1):
            if t <= n + j:
                got = out[j].float().cpu()
                assert (got - want.float()[None, :]).abs().max() <= 2 ** -7 * want.float().abs().max() + 1e-6, (t, j)
        L.k_pool.copy_(kp); L.k_new.copy_(kn)


def _scale_logical_pages(b, pool, factor_of_position):
    """Multiplies the keys (or values) of every request's logical position t by factor_of_position(i, t) (a power of
    two, so bf16 stays exact), page by page through the block table."""
    bs = b.block_size
    for i in range(b.batch):
        for p in range(-(-int(b.seq_lens[i]) // bs)):
            f = factor_of_position(i, p * bs)
            if f != 1.0:
                pool[b.block_table[i, p]] = (pool[b.block_table[i, p]].float() * f).to(torch.bfloat16)


@pytest.mark.parametrize("impl_i", [0, 1])
@pytest.mark.parametrize("D,Hq,dl", [(64, 64, [16, 3, 9, 0]), (64, 16, [15, 7, 2, 0]), (128, 32, [8, 3, 0, 6])])
@pytest.mark.parametrize("factors", [(8.0, 64.0), (1.0, 512.0), (0.125, 1.0)])
def test_scores_that_outgrow_their_reference(bnd, impl_i, D, Hq, dl, factors):
    """Keys whose scale jumps in the middle of the context: the later tiles' scores lie tens to thousands of log2 units
    above (or, shrinking, below) the running reference the first tiles set.  Covers references that move after a
    tile's weights were computed and weights that overflow fp32 before they do."""
    seq = [3000, 700, 1400, 129]
    b = workloads.make_batch("t", seed=77, seq_lens=seq, draft_lens=dl, num_q_heads=Hq, num_kv_heads=8, head_dim=D,
                             vocab=8, with_logits=False)
    f1, f2 = factors
    cut = lambda i, t: f2 if t >= (2 * seq[i]) // 3 // 128 * 128 + 48 else (f1 if t >= seq[i] // 3 else 1.0)
    _scale_logical_pages(b, b.layers[0].k_pool, cut)
    r = run_attn(bnd, b, impls(bnd)[impl_i])
    if r is None:
        pytest.skip("tensor-core kernel does not cover this shape")
    _, out, lse = r
    want, want_lse = oracle_attn(b)
    mx, mean, rel = attn_errors(out, want)
    assert mx <= ATTN_MAX_ABS and mean <= ATTN_MEAN_ABS and rel <= ATTN_REL_FRO, (mx, mean, rel)
    # (an lse of several hundred carries fp32 rounding of its own: 1e-3 absolute plus 2e-6 relative)
    assert (np.abs(lse.double().cpu().numpy() - want_lse) <= LSE_ABS + 2e-6 * np.abs(want_lse)).all()


@pytest.mark.parametrize("impl_i", [0, 1])
@pytest.mark.parametrize("D,Hq,window", [(64, 64, 0), (64, 64, 128), (128, 32, 0), (128, 32, 128)])
def test_slots_no_request_can_see_may_hold_anything(bnd, impl_i, D, Hq, window):
    """A real cache is not initialised: the tail of a request's last page, pages that no request owns and slots of
    rolled-back drafts hold whatever was there before.  Fill every such slot of both pools with NaN and Inf bit patterns:
    output and lse must be what they are with finite tails, bit for bit, and match the oracle.  Lengths are chosen so
    that n + k + 1 is neither a multiple of 128 nor of the page size; one request is long enough to be split."""
    seq = [70, 397, 40000 + 5, 1027, 255]
    dl = [3, 9, 5, 0, 6] if D == 128 else [3, 16, 5, 0, 11]
    g = torch.Generator().manual_seed(3)
    kinds = [workloads.LayerKind(window=window, sinks=torch.randn(Hq, generator=g))]
    b = workloads.make_batch("t", seed=88, seq_lens=seq, draft_lens=dl, num_q_heads=Hq, num_kv_heads=8, head_dim=D,
                             vocab=8, kinds=kinds, with_logits=False)
    r = run_attn(bnd, b, impls(bnd)[impl_i])
    if r is None:
        pytest.skip("tensor-core kernel does not cover this shape")
    _, out0, lse0 = r
    out0, lse0 = out0.clone(), lse0.clone()
    want, want_lse = oracle_attn(b)
    check_attn(out0, lse0, want, want_lse)
    # poison: every slot at a position >= n_i + k_i + 1 of a request's pages, and every page nobody owns
    L = b.layers[0]
    bs = b.block_size
    owned = np.zeros(L.k_pool.shape[0], bool)
    poison = torch.tensor([float("nan"), float("inf"), -float("inf"), float("nan")]).to(torch.bfloat16)
    for i in range(b.batch):
        end = int(b.seq_lens[i] + b.draft_lens[i] + 1)
        pages = -(-end // bs)
        owned[b.block_table[i, :pages]] = True
        if end % bs:
            for pool in (L.k_pool, L.v_pool):
                tail = pool[b.block_table[i, pages - 1], :, end % bs:, :]
                tail.copy_(poison[torch.arange(tail.numel()) % 4].reshape(tail.shape))
    for pool in (L.k_pool, L.v_pool):
        free = torch.as_tensor(np.nonzero(~owned)[0])
        if len(free):
            pool[free] = float("nan")
    r = run_attn(bnd, b, impls(bnd)[impl_i])
    _, out1, lse1 = r
    assert torch.equal(out0.view(torch.int16), out1.view(torch.int16))
    assert torch.equal(lse0.view(torch.int32), lse1.view(torch.int32))


def _check_sampled(bnd, b, vs, band=1e-5):
    """Applies the band rule; returns (#positions inside the band, #positions)."""
    ref = oracle_accept(b, want_ratios=True)
    got_a = vs.accept_len.cpu().numpy()
    got_t = vs.out_tokens.cpu().numpy()
    _, cu_d = cu(b.draft_lens)
    cu_q, _ = cu(b.draft_lens)
    in_band = 0
    force = np.full(b.batch, -1, np.int32)
    for i in range(b.batch):
        if got_a[i] != ref["accept_len"][i]:
            j = min(got_a[i], ref["accept_len"][i])                         # first position decided differently
            ratio = ref["ratios"][cu_d[i] + j]
            assert abs(ratio - float(b.u[cu_d[i] + j])) <= band, (i, j, ratio, b.u[cu_d[i] + j])
            in_band += 1
            force[i] = got_a[i]
    if in_band:
        ref = oracle_accept(b, force_accept=force)
    assert np.array_equal(got_a, ref["accept_len"])
    logits = b.logits.cpu().numpy()
    dp = None if b.draft_probs is None else b.draft_probs.cpu().numpy()
    exact = 0
    for i in range(b.batch):
        a, k = int(got_a[i]), int(b.draft_lens[i])
        assert np.array_equal(got_t[i, :a], ref["out_tokens"][i, :a])
        assert (got_t[i, a + 1:] == -1).all()
        v = int(got_t[i, a])
        if v == ref["out_tokens"][i, a]:
            exact += 1
            continue
        T = float(b.temperature[i]) if b.temperature is not None else 0.0
        assert T > 0, "greedy extra token must be exact"
        lo, hi, S, rv = oracle.recovery_interval(k, a, logits[cu_q[i] + a], b.vocab,
                                                 dp[cu_d[i] + a] if (dp is not None and a < k) else None,
                                                 int(b.draft_tokens[cu_d[i] + a]) if a < k else -1, T, v)
        wS = float(b.w[cu_q[i] + a]) * S
        assert rv > 0 and lo - band * S <= wS < hi + band * S, (i, v, lo, hi, wS)
    return in_band, b.total_d, exact


@pytest.mark.parametrize("dense", [True, False])
@pytest.mark.parametrize("vocab,ld", [(50, 50), (4099, 4104), (20000, 20000)])
def test_sampled_acceptance(bnd, dense, vocab, ld):
    b = workloads.make_batch("t", seed=77 + vocab, seq_lens=[20] * 48, draft_lens=list(np.arange(48) % 7),
                             num_q_heads=8, num_kv_heads=2, head_dim=128, vocab=vocab, ld=ld, logit_std=2.0,
                             match="sample", temperature=0.7, dense_draft_probs=dense, k_max=6)
    # mixed batch: every fifth request is greedy
    b.temperature[::5] = 0.0
    vs = bnd.VerifyStep(b)
    vs.plan_step()
    vs.accept()
    assert bnd.as_plan_check(vs.plan) == 0
    in_band, total, exact = _check_sampled(bnd, b, vs)
    assert in_band <= max(1, 1e-4 * total)
    assert exact >= b.batch - 1


@pytest.mark.parametrize("dense", [True, False])
@pytest.mark.parametrize("seed,step", [(0, 0), (0x123456789ABCDEF, 41), (5, (1 << 40) + 3)])
def test_seeded_acceptance_draws_the_oracles_uniforms(bnd, dense, seed, step):
    """as_accept_seeded: the kernels draw u and w themselves (Philox4x32-10); the oracle draws the same
    numbers with its own implementation of the generator and verifies with them."""
    b = workloads.make_batch("t", seed=900 + step % 97, seq_lens=[20] * 40, draft_lens=list(np.arange(40) % 7),
                             num_q_heads=8, num_kv_heads=2, head_dim=128, vocab=4099, ld=4104, logit_std=2.0,
                             match="sample", temperature=0.7, dense_draft_probs=dense, k_max=6)
    b.temperature[::5] = 0.0
    u, w_req = oracle.philox_uniforms(seed, step, b.draft_lens)
    cu_q, _ = cu(b.draft_lens)
    w = np.zeros(b.total_q, dtype=np.float32)               # the oracle reads w at row a_i: the same draw for every row
    for i in range(b.batch):
        w[cu_q[i]:cu_q[i + 1]] = w_req[i]
    b.u, b.w = u, w
    vs = bnd.VerifyStep(b)
    vs.plan_step()
    to_i64 = lambda x: x - (1 << 64) if x >= (1 << 63) else x
    rng = torch.tensor([to_i64(seed), to_i64(step)], dtype=torch.int64, device="cuda")
    bnd.as_accept_seeded(vs.plan, vs.logits, b.vocab, vs.draft_tokens, vs.draft_probs, vs.temperature, rng,
                         vs.accept_len, vs.out_tokens)
    assert bnd.as_plan_check(vs.plan) == 0
    in_band, total, exact = _check_sampled(bnd, b, vs)
    assert in_band <= max(1, 1e-4 * total)
    assert exact >= b.batch - 1
    # the passed-in path with the same numbers gives the same answer bit for bit
    a1, t1 = vs.accept_len.clone(), vs.out_tokens.clone()
    vs.u, vs.w = torch.as_tensor(u, device="cuda"), torch.as_tensor(w, device="cuda")
    vs.rebind()
    vs.accept()
    assert torch.equal(a1, vs.accept_len) and torch.equal(t1, vs.out_tokens)


@pytest.mark.parametrize("vocab,ld", [(7, 7), (4096, 4096), (151936, 151936), (5001, 5003)])
def test_greedy_acceptance_exact(bnd, vocab, ld):
    b = workloads.make_batch("t", seed=vocab, seq_lens=[20] * 16, draft_lens=list(np.arange(16) % 9), num_q_heads=8,
                             num_kv_heads=2, head_dim=128, vocab=vocab, ld=ld, logit_std=2.0, match_p=0.7, k_max=8)
    # plant ties, NaN and infinities: ties must go to the lowest index, NaN never wins
    z = b.logits
    z[0, :] = 1.0
    z[1, vocab - 1] = float("inf"); z[1, 0] = float("inf")
    z[2, 3 % vocab] = float("nan")
    z[3, :] = float("nan")
    mx = z[4, :vocab].max(); z[4, vocab // 2] = mx; z[4, vocab - 1] = mx
    if ld > vocab:
        z[:, vocab:] = 1e30                                                  # padding columns are never read
    vs = bnd.VerifyStep(b)
    vs.plan_step()
    vs.accept()
    assert bnd.as_plan_check(vs.plan) == 0
    ref = oracle_accept(b)
    assert np.array_equal(vs.accept_len.cpu().numpy(), ref["accept_len"])
    assert np.array_equal(vs.out_tokens.cpu().numpy(), ref["out_tokens"])


def test_commit_rollback_and_page_assignment(bnd):
    """as_plan hands out tentative pages from a free list; commit returns the unused ones in order."""
    bs, B, kmax = 16, 9, 8
    rng = np.random.default_rng(1)
    seq = np.array([0, 1, 15, 16, 17, 31, 32, 100, 255], np.int32)
    dl = np.array([8, 0, 1, 8, 8, 0, 3, 8, 1], np.int32)
    b = workloads.make_batch("t", seed=9, seq_lens=seq, draft_lens=dl, num_q_heads=8, num_kv_heads=2, head_dim=64,
                             vocab=8, block_size=bs, with_logits=False, k_max=kmax)
    held = -(-seq // bs)
    need = -(-(seq + dl + 1) // bs)
    # strip the tentative pages out of the generator's table and offer them (shuffled) as the free list
    table = b.block_table.copy()
    free = []
    for i in range(B):
        free += list(table[i, held[i]:need[i]]); table[i, held[i]:] = -1
    free = [int(x) for x in rng.permutation(free)]
    vs = bnd.VerifyStep(b)
    vs.block_table.copy_(torch.as_tensor(table))
    taken = bnd.as_plan(vs.plan, seq, dl, vs.block_table, free)
    assert taken == int((need - held).sum())
    want_table = table.copy()
    at = 0
    for i in range(B):
        for l in range(held[i], need[i]):
            want_table[i, l] = free[at]; at += 1
    torch.cuda.synchronize()
    assert np.array_equal(vs.block_table.cpu().numpy(), want_table)
    with pytest.raises(bnd.AsError) as e:
        bnd.as_plan(vs.plan, seq, dl, vs.block_table, free[:2])
    assert e.value.status == bnd.AS_ERR_INVALID_ARG
    vs.block_table.copy_(torch.as_tensor(table))
    bnd.as_plan(vs.plan, seq, dl, vs.block_table, free)
    b.block_table = want_table
    for trial in range(3):
        vs.attn(0)                                                           # tentative append of all k_i + 1 rows
        a = np.minimum(rng.integers(0, kmax + 1, size=B), dl).astype(np.int32)
        vs2_table = torch.as_tensor(want_table).cuda()
        seq_dev = torch.as_tensor(seq).cuda()
        vs.accept_len.copy_(torch.as_tensor(a))
        bnd.as_kv_commit(vs.plan, vs.accept_len, seq_dev, vs2_table, vs.freed, vs.freed_count,
                         bnd.AS_COMMIT_SCRUB if trial % 2 == 0 else 0, vs.layers[0].k_pool, vs.layers[0].v_pool)
        assert bnd.as_plan_check(vs.plan) == 0
        seq2, bt2, kp, vp, freed = oracle_commit(b, a, scrub=trial % 2 == 0)
        assert np.array_equal(seq_dev.cpu().numpy(), seq2)
        assert np.array_equal(vs2_table.cpu().numpy(), bt2)
        assert np.array_equal(vs.freed.cpu().numpy()[:int(vs.freed_count.item())], freed)
        gk = np_bits(vs.layers[0].k_pool)
        for i in range(B):
            upto = int(seq2[i]) if trial % 2 else min(-(-int(seq2[i]) // bs) * bs, int(seq[i] + dl[i] + 1))
            assert np.array_equal(gather_logical(gk, bt2[i], upto, bs), gather_logical(kp, bt2[i], upto, bs))
        # as_kv_commit consumed the plan: the next step must plan again
        with pytest.raises(bnd.AsError):
            bnd.as_kv_commit(vs.plan, vs.accept_len, seq_dev, vs2_table, vs.freed, vs.freed_count)
        bnd.as_plan(vs.plan, seq, dl, torch.as_tensor(want_table).cuda(), None)


def test_commit_leaves_table_entries_beyond_the_step_alone(bnd):
    """Pages a scheduler reserved further out in a request's block-table row are not the step's to release: commit
    frees only logical pages in [ceil(n'/bs), ceil((n+k+1)/bs)) and leaves later entries where they are."""
    b = workloads.make_batch("t", seed=12, seq_lens=[30, 170, 62], draft_lens=[5, 2, 8], num_q_heads=8, num_kv_heads=2,
                             head_dim=64, vocab=8, block_size=16, with_logits=False, k_max=8)
    need = -(-(b.seq_lens + b.draft_lens + 1) // 16)
    used = set(int(x) for x in b.block_table.ravel() if x >= 0)
    spare = [p for p in range(b.num_blocks) if p not in used]
    assert len(spare) >= 4
    b.block_table[0, need[0]:need[0] + 2] = spare[:2]           # live entries past request 0's and 2's last position
    b.block_table[2, need[2]] = spare[2]
    for a in ([0, 0, 0], [5, 1, 3], [2, 2, 8]):
        vs = bnd.VerifyStep(b)
        vs.plan_step()
        vs.attn(0)
        vs.accept_len.copy_(torch.as_tensor(np.array(a, np.int32)))
        vs.commit()
        assert bnd.as_plan_check(vs.plan) == 0
        seq2, bt2, _, _, freed = oracle_commit(b, a)
        assert np.array_equal(vs.seq_lens.cpu().numpy(), seq2)
        assert np.array_equal(vs.block_table.cpu().numpy(), bt2)
        assert list(bt2[0, need[0]:need[0] + 2]) == spare[:2] and bt2[2, need[2]] == spare[2]
        assert np.array_equal(vs.freed.cpu().numpy()[:int(vs.freed_count.item())], freed)
        assert not set(freed.tolist()) & set(spare)


def test_device_faults_are_flagged_not_trapped(bnd):
    b = workloads.make_batch("t", seed=4, seq_lens=[40, 40], draft_lens=[2, 2], num_q_heads=8, num_kv_heads=2,
                             head_dim=128, vocab=64, block_size=16, k_max=2)
    vs = bnd.VerifyStep(b)
    vs.block_table[1, 1] = b.num_blocks + 5            # page id outside the pool
    vs.draft_tokens[0] = 64                            # token outside the vocabulary
    vs.plan_step()
    vs.attn(0)
    vs.accept()
    vs.accept_len[1] = 7                               # accepted length > k_i
    vs.commit()
    flags = bnd.as_plan_check(vs.plan, raise_on_flag=False)
    assert flags & bnd.AS_FLAG_BAD_PAGE and flags & bnd.AS_FLAG_BAD_TOKEN and flags & bnd.AS_FLAG_BAD_ACCEPT
    assert int(vs.seq_lens[1]) == 40 + 2 + 1           # clamped to k_i
    assert bnd.as_plan_check(vs.plan) == 0             # the word was cleared; the context is still usable
    out = torch.zeros(4, device="cuda") + 1
    assert float(out.sum()) == 4.0


@pytest.mark.parametrize("D,Hq,stall", [(128, 32, 3), (128, 32, 0), (64, 64, 5), (64, 64, 0)])
def test_a_wait_that_runs_out_is_reported_and_leaves_the_plan_usable(bnd, D, Hq, stall):
    """Failure detection without a fault: the test hook tells every CTA's copy producers to stop after `stall` tiles
    and shortens the kernels' wait limit to 3 ms, so the waits behind the missing copies run out.  The kernel must
    return by itself, as_plan_check must report AS_ERR_TIMEOUT with AS_FLAG_WAIT_CAP and a bit naming a wait, and the
    next ordinary step on the same plan, workspace and pools must equal a step on a fresh plan bit for bit."""
    b = workloads.make_batch("t", seed=21, seq_lens=[3000, 900, 5000, 129], draft_lens=[4, 8, 0, 6], num_q_heads=Hq,
                             num_kv_heads=8, head_dim=D, vocab=8, with_logits=False)
    fresh = bnd.VerifyStep(b, attn_impl=bnd.AS_ATTN_TC)
    fresh.plan_step(); fresh.attn(0)
    assert bnd.as_plan_check(fresh.plan) == 0
    want_out, want_lse = fresh.out[0].clone(), fresh.lse[0].clone()

    vs = bnd.VerifyStep(b, attn_impl=bnd.AS_ATTN_TC)
    vs.plan_step()
    bnd.as_plan_set_test_stall(vs.plan, 3_000_000, stall)
    vs.attn(0)
    with pytest.raises(bnd.AsError) as e:
        bnd.as_plan_check(vs.plan)
    assert e.value.status == bnd.AS_ERR_TIMEOUT
    vs.plan_step(); vs.attn(0)                                 # still stalling: the flags say which waits gave up
    flags = bnd.as_plan_check(vs.plan, raise_on_flag=False)
    assert flags & bnd.AS_FLAG_WAIT_CAP and flags >> 8, hex(flags)
    bnd.as_plan_set_test_stall(vs.plan, 0, -1)
    vs.plan_step(); vs.attn(0)
    assert bnd.as_plan_check(vs.plan) == 0
    assert torch.equal(vs.out[0].view(torch.int16), want_out.view(torch.int16))
    assert torch.equal(vs.lse[0].view(torch.int32), want_lse.view(torch.int32))


def test_empty_batch_and_argument_errors(bnd):
    b = workloads.tiny()
    vs = bnd.VerifyStep(b)
    assert bnd.as_plan(vs.plan, [], [], vs.block_table) == 0
    vs.attn(0); vs.accept()
    with pytest.raises(bnd.AsError) as e:
        bnd.as_plan(vs.plan, [10], [9], vs.block_table)                     # k > max_draft
    assert e.value.status == bnd.AS_ERR_INVALID_ARG
    with pytest.raises(bnd.AsError) as e:
        vs.attn(0)                                                           # failed plan leaves nothing planned
    assert e.value.status == bnd.AS_ERR_INVALID_ARG
    vs.plan_step()
    with pytest.raises(bnd.AsError):
        bnd.as_verify_attn(vs.plan, 3, vs.layers[0].q, vs.layers[0].k_new, vs.layers[0].v_new, vs.layers[0].k_pool,
                           vs.layers[0].v_pool, vs.block_table, vs.out[0])   # kind out of range
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(bnd.AsError) as e:
        bnd.as_plan_bind(vs.plan, small)
    assert e.value.status == bnd.AS_ERR_WORKSPACE


def test_more_items_per_cta_than_the_shared_memory_mirror_holds(bnd):
    """12000 one-tile (request, kv-head) pairs on 148 CTAs: about 81 work items per CTA, more than the 64
    the kernel mirrors in shared memory, so the tail of every CTA's list comes from global memory."""
    rng = np.random.default_rng(3)
    B = 1500
    seq = rng.integers(1, 100, size=B).astype(np.int32)
    dl = rng.integers(0, 4, size=B).astype(np.int32)
    b = workloads.make_batch("t", seed=12, seq_lens=seq, draft_lens=dl, num_q_heads=16, num_kv_heads=8, head_dim=128,
                             vocab=8, with_logits=False, k_max=3)
    r = run_attn(bnd, b, bnd.AS_ATTN_TC)
    assert r is not None
    vs, out, lse = r
    assert bnd.as_plan_stats(vs.plan, 0)["num_items"] >= 148 * 70
    want, want_lse = oracle_attn(b)
    check_attn(out, lse, want, want_lse)


def test_results_are_bitwise_reproducible(bnd):
    b = workloads.make_batch("t", seed=8, seq_lens=[3000, 200, 1500, 90], draft_lens=[4, 8, 0, 2], num_q_heads=32,
                             num_kv_heads=8, head_dim=128, vocab=8, with_logits=False)
    outs = []
    for rep in range(3):
        vs = bnd.VerifyStep(b)
        vs.plan_step(); vs.attn(0)
        torch.cuda.synchronize()
        outs.append((vs.out[0].clone(), vs.lse[0].clone()))
    for o, l in outs[1:]:
        assert torch.equal(o, outs[0][0]) and torch.equal(l, outs[0][1])


@pytest.mark.parametrize("D,Hq,kmax,dl", [(64, 64, 16, [16, 3, 0, 9, 12]), (64, 64, 9, [9, 3, 0, 9, 5]), (128, 32, 8, [8, 3, 0, 8, 5])])
def test_results_do_not_depend_on_what_memory_held_before(bnd, D, Hq, kmax, dl):
    """Bit-reproducibility: the first call on a freshly bound, poisoned workspace (and whatever the previous kernels
    left in shared and tensor memory) gives the same bits as the calls after it.  Tiles with fewer rows than the
    hardware tile hold rows that belong to no request; nothing they compute may steer the others."""
    b = workloads.make_batch("t", seed=41, seq_lens=[5000, 300, 127, 20000, 64], draft_lens=dl, num_q_heads=Hq, num_kv_heads=8,
                             head_dim=D, vocab=8, with_logits=False, k_max=kmax)
    vs = bnd.VerifyStep(b, attn_impl=bnd.AS_ATTN_TC)
    ws = torch.full_like(vs.ws, 0xFF)
    bnd.as_plan_bind(vs.plan, ws); vs.ws = ws
    vs.plan_step(); vs.attn(0); torch.cuda.synchronize()
    first_out, first_lse = vs.out[0].clone(), vs.lse[0].clone()
    for _ in range(2):
        vs.attn(0); torch.cuda.synchronize()
        assert torch.equal(vs.out[0][:b.total_q], first_out[:b.total_q]) and torch.equal(vs.lse[0][:b.total_q], first_lse[:b.total_q])
    assert bnd.as_plan_check(vs.plan) == 0
    want, want_lse = oracle_attn(b)
    check_attn(first_out[:b.total_q], first_lse[:b.total_q], want, want_lse)
