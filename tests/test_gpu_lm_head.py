"""as_accept_lm_head(): greedy acceptance from hidden states through the output projection on the tensor cores,
against the oracle's projection (fp64) followed by its greedy acceptance.  The kernel accumulates in fp32 in the
tensor cores' own order, so a row whose two largest logits are closer than `BAND` may legitimately go either way:
such rows are counted, must be few, and every disagreement must trace back to one of them."""
import copy

import numpy as np
import pytest
import torch

import oracle
from paper_2608_24004_b200 import workloads
from helpers import cu, oracle_accept
from test_gpu_parity import _check_sampled

pytestmark = pytest.mark.gpu
BAND = 2e-3            # logits are O(2) here; fp32 accumulation over <= 1024 products stays far below this


@pytest.fixture(scope="module")
def bnd():
    from paper_2608_24004_b200 import build as as_build
    as_build.build_library()
    from paper_2608_24004_b200 import binding
    return binding


def _setup(seed, seq, dl, H, V, match_p=0.6):
    """A batch whose logits are the oracle's projection of seeded hidden states; drafts hit its argmax w.p. match_p."""
    A = workloads.make_batch("lm", seed=seed, seq_lens=seq, draft_lens=dl, num_q_heads=8, num_kv_heads=2, head_dim=128, vocab=V,
                             with_logits=False, k_max=max(dl))
    g = torch.Generator().manual_seed(seed + 9)
    hidden = torch.randn((A.total_q, H), generator=g).to(torch.bfloat16)
    weight = (torch.randn((V, H), generator=g) * (2.0 / H ** 0.5)).to(torch.bfloat16)
    logits = oracle.lm_head(oracle.bf16_bits(hidden), oracle.bf16_bits(weight))
    A = copy.copy(A)
    A.logits = torch.as_tensor(logits.astype(np.float32))
    rng = np.random.default_rng(seed)
    cu_q, _ = cu(A.draft_lens)
    toks = []
    for i in range(A.batch):
        for j in range(int(A.draft_lens[i])):
            tgt = int(np.argmax(logits[cu_q[i] + j]))
            toks.append(tgt if rng.random() < match_p else int((tgt + 1 + rng.integers(0, V - 1)) % V))
    A.draft_tokens = np.asarray(toks, dtype=np.int32)
    return A, hidden, weight, logits


def _run(bnd, A, hidden, weight, fixed=False):
    vs = bnd.VerifyStep(A)
    if fixed:
        bnd.as_plan_set_fixed_launch(vs.plan, True)
        pad = torch.zeros((A.batch * (A.k_max + 1), hidden.shape[1]), dtype=torch.bfloat16)
        pad[:hidden.shape[0]] = hidden
        hidden = pad
    vs.plan_step()
    bnd.as_accept_lm_head(vs.plan, hidden.cuda().contiguous(), weight.cuda().contiguous(), vs.draft_tokens, vs.accept_len,
                          vs.out_tokens)
    torch.cuda.synchronize()
    assert bnd.as_plan_check(vs.plan) == 0
    return vs.accept_len.cpu().numpy()[:A.batch], vs.out_tokens.cpu().numpy()[:A.batch]


def _compare(A, logits, got_len, got_tok):
    acc = oracle_accept(A)
    top2 = np.sort(logits, axis=1)[:, -2:]
    near = (top2[:, 1] - top2[:, 0]) < BAND                       # rows the two sides may decide differently
    cu_q, _ = cu(A.draft_lens)
    bad = 0
    for i in range(A.batch):
        same = got_len[i] == acc["accept_len"][i] and np.array_equal(got_tok[i], acc["out_tokens"][i])
        if not same:
            judged = slice(cu_q[i], cu_q[i] + min(got_len[i], acc["accept_len"][i]) + 1)
            assert near[judged].any(), (i, got_len[i], acc["accept_len"][i])
            bad += 1
    return bad, int(near.sum())


CASES = [
    # (seed, seq_lens, draft_lens, H, V)
    (1, [100, 20, 300], [4, 0, 6], 256, 1000),                    # one row tile, four vocabulary tiles (the last ragged)
    (2, [50] * 40, [5] * 40, 512, 4099),                          # 240 rows: two row tiles, V not a multiple of anything
    (3, [10, 10], [3, 2], 64, 200),                               # a single K block, vocabulary smaller than a tile
    (4, [700] * 9, [16] * 9, 1024, 2560),                         # 153 rows, V an exact multiple of the tile
]


@pytest.mark.parametrize("fixed", [False, True])
@pytest.mark.parametrize("case", CASES)
def test_greedy_acceptance_from_hidden_states(bnd, case, fixed):
    seed, seq, dl, H, V = case
    A, hidden, weight, logits = _setup(seed, seq, dl, H, V)
    got_len, got_tok = _run(bnd, A, hidden, weight, fixed=fixed)
    bad, near = _compare(A, logits, got_len, got_tok)
    assert near <= max(2, A.total_q // 20), near                   # the band is narrow
    assert bad <= near


def test_exact_inputs_ties_and_nan(bnd):
    """Small integers: every product and sum is exact in fp32, so the result must equal the oracle's exactly, ties
    included (equal columns -> the lowest wins; -0 ties with +0; a NaN column never wins)."""
    seq, dl, H, V = [5, 9, 0], [3, 4, 2], 128, 600
    A = workloads.make_batch("lm_x", seed=5, seq_lens=seq, draft_lens=dl, num_q_heads=8, num_kv_heads=2, head_dim=128, vocab=V,
                             with_logits=False, k_max=4)
    rng = np.random.default_rng(5)
    hidden = torch.as_tensor(rng.integers(-3, 4, size=(A.total_q, H)), dtype=torch.float32).to(torch.bfloat16)
    weight = torch.as_tensor(rng.integers(-2, 3, size=(V, H)), dtype=torch.float32).to(torch.bfloat16)
    weight[300] = weight[17]                                       # duplicate columns: ties wherever 17 is the maximum
    weight[555] = weight[17]
    weight[42] = float("nan")
    weight[299] = 0.0                                              # logit +0 / -0 depending on nothing: must tie with other zeros
    logits = oracle.lm_head(oracle.bf16_bits(hidden), oracle.bf16_bits(weight))
    logits = np.where(np.isnan(logits), -np.inf, logits)
    A = copy.copy(A)
    A.logits = torch.as_tensor(logits.astype(np.float32))
    cu_q, _ = cu(A.draft_lens)
    toks = []
    for i in range(A.batch):
        for j in range(dl[i]):
            tgt = int(np.argmax(logits[cu_q[i] + j]))               # numpy's argmax is the lowest index too
            toks.append(tgt if (i + j) % 3 else (tgt + 1) % V)
    A.draft_tokens = np.asarray(toks, dtype=np.int32)
    got_len, got_tok = _run(bnd, A, hidden, weight)
    acc = oracle_accept(A)
    assert np.array_equal(got_len, acc["accept_len"])
    assert np.array_equal(got_tok, acc["out_tokens"])
    # make the maximum of one row sit in the duplicated columns and check which one is reported
    hidden2 = hidden.clone()
    hidden2[0] = (weight[17].float() * 3).to(torch.bfloat16)       # <h, w_17> = 3 |w_17|^2: far above every other column
    logits2 = oracle.lm_head(oracle.bf16_bits(hidden2), oracle.bf16_bits(weight))
    logits2 = np.where(np.isnan(logits2), -np.inf, logits2)
    assert int(np.argmax(logits2[0])) == 17 and logits2[0, 17] == logits2[0, 300] == logits2[0, 555]
    B = copy.copy(A)
    B.logits = torch.as_tensor(logits2.astype(np.float32))
    got_len2, got_tok2 = _run(bnd, B, hidden2, weight)
    acc2 = oracle_accept(B)
    assert np.array_equal(got_len2, acc2["accept_len"]) and np.array_equal(got_tok2, acc2["out_tokens"])


def test_full_size_projection_row_argmax(bnd):
    """The bench's own projection size (hidden 4096, vocabulary 151936: 594 vocabulary tiles, 64 K blocks) on 24 rows
    without drafts, so that out_tokens[i][0] is row i's argmax itself; the oracle computes those 24 rows in fp64."""
    H, V, B = 4096, 151936, 24
    A = workloads.make_batch("lm_full", seed=7, seq_lens=[40] * B, draft_lens=[0] * B, num_q_heads=8, num_kv_heads=2, head_dim=128,
                             vocab=V, with_logits=False, k_max=0)
    g = torch.Generator().manual_seed(70)
    hidden = torch.randn((B, H), generator=g).to(torch.bfloat16)
    weight = (torch.randn((V, H), generator=g) * (2.0 / H ** 0.5)).to(torch.bfloat16)
    logits = oracle.lm_head(oracle.bf16_bits(hidden), oracle.bf16_bits(weight))
    vs = bnd.VerifyStep(A)
    vs.plan_step()
    bnd.as_accept_lm_head(vs.plan, hidden.cuda(), weight.cuda(), vs.draft_tokens, vs.accept_len, vs.out_tokens)
    torch.cuda.synchronize()
    assert bnd.as_plan_check(vs.plan) == 0
    got = vs.out_tokens.cpu().numpy()[:B, 0]
    assert (vs.accept_len.cpu().numpy()[:B] == 0).all()
    want = np.argmax(logits, axis=1)
    top2 = np.sort(logits, axis=1)[:, -2:]
    near = (top2[:, 1] - top2[:, 0]) < BAND
    for i in range(B):
        if got[i] != want[i]:
            assert near[i] and abs(logits[i, got[i]] - top2[i, 1]) < BAND, (i, got[i], want[i])
    assert int((got != want).sum()) <= int(near.sum()) <= 2


# ---- rejection sampling from hidden states (as_accept_lm_head_sampled) ----------------------------------------------
# The accept ratio min(1, p[d] / q[d]) is built from logits that the tensor cores accumulate in fp32 in their own order:
# a logit of size O(2) over H <= 1024 products carries about 1e-6 of error, p[d] (a ratio of exponentials of z / T) a few
# 1e-6 relative, so a decision may legitimately differ from the oracle's where the oracle's ratio lies within SAMPLED_BAND
# of the uniform; such positions are counted, must be rare, and the oracle is re-run with the decision forced so that the
# rest of the request is still checked exactly.  The extra token is accepted when w * S lies in its CDF step widened by
# the same band.
SAMPLED_BAND = 1e-4


def _setup_sampled(seed, seq, dl, H, V, T, dense):
    A = workloads.make_batch("lm", seed=seed, seq_lens=seq, draft_lens=dl, num_q_heads=8, num_kv_heads=2, head_dim=128, vocab=V,
                             with_logits=False, k_max=max(dl))
    g = torch.Generator().manual_seed(seed + 9)
    hidden = torch.randn((A.total_q, H), generator=g).to(torch.bfloat16)
    weight = (torch.randn((V, H), generator=g) * (2.0 / H ** 0.5)).to(torch.bfloat16)
    logits = torch.as_tensor(oracle.lm_head(oracle.bf16_bits(hidden), oracle.bf16_bits(weight)).astype(np.float32))
    A = copy.copy(A)
    A.logits = logits
    cu_q, _ = cu(A.draft_lens)
    rows = np.concatenate([cu_q[i] + np.arange(A.draft_lens[i]) for i in range(A.batch)]).astype(np.int64)
    temp = np.full(A.batch, T, np.float32)
    temp[A.batch - 1] = 0.0                                         # the last request is greedy: mixed batches are allowed
    t_rows = np.repeat(np.maximum(temp, 0.5), A.draft_lens)
    zd = logits[torch.as_tensor(rows)] + torch.randn((len(rows), V), generator=g)
    qd = torch.softmax(zd / torch.as_tensor(t_rows)[:, None], dim=-1)
    A.draft_tokens = torch.multinomial(qd, 1, generator=g).squeeze(1).numpy().astype(np.int32)
    A.draft_probs = qd.contiguous() if dense else None
    A.temperature = temp
    rng = np.random.Generator(np.random.Philox(seed + 3))
    A.u = rng.random(A.total_d, dtype=np.float32)
    A.w = rng.random(A.total_q, dtype=np.float32)
    return A, hidden, weight


@pytest.mark.parametrize("dense", [True, False])
@pytest.mark.parametrize("seed,seq,dl,H,V,T", [
    (21, [100, 20, 300, 50], [4, 0, 6, 3], 256, 1000, 0.7),          # one row tile, four vocabulary tiles (the last ragged)
    (22, [64] * 40, [6] * 40, 512, 5001, 0.7),                       # three row tiles, twenty vocabulary tiles
    (23, [30] * 9, [8, 0, 1, 8, 8, 0, 3, 8, 1], 1024, 20000, 1.3),
])
def test_sampled_acceptance_from_hidden_states(bnd, seed, seq, dl, H, V, T, dense):
    A, hidden, weight = _setup_sampled(seed, seq, dl, H, V, T, dense)
    vs = bnd.VerifyStep(A)
    vs.plan_step()
    scratch = torch.empty(bnd.as_accept_lm_head_scratch_bytes(vs.plan, H, V), dtype=torch.uint8, device="cuda")
    bnd.as_accept_lm_head_sampled(vs.plan, hidden.cuda().contiguous(), weight.cuda().contiguous(), vs.draft_tokens, vs.draft_probs,
                                  vs.temperature, vs.u, vs.w, None, scratch, vs.accept_len, vs.out_tokens)
    torch.cuda.synchronize()
    assert bnd.as_plan_check(vs.plan) == 0
    in_band, total, exact = _check_sampled(bnd, A, vs, band=SAMPLED_BAND)
    assert in_band <= max(1, 0.02 * total), (in_band, total)
    assert exact >= 0.9 * A.batch, exact
    # and the same decisions as as_accept on the materialised fp32 logits of the oracle, outside the band
    vs2 = bnd.VerifyStep(A)
    vs2.plan_step(); vs2.accept()
    same = (vs2.accept_len == vs.accept_len).float().mean().item()
    assert same >= 0.9, same


def test_full_size_sampled_acceptance_from_hidden_states(bnd):
    """The R1-shaped projection (hidden 4096, vocabulary 128256: 501 vocabulary tiles, 64 K blocks), six requests of six
    drafts at temperature 0.7 with dense draft probabilities; the oracle projects those 42 rows in fp64."""
    A, hidden, weight = _setup_sampled(41, [40] * 6, [6] * 6, 4096, 128256, 0.7, True)
    vs = bnd.VerifyStep(A)
    vs.plan_step()
    scratch = torch.empty(bnd.as_accept_lm_head_scratch_bytes(vs.plan, 4096, 128256), dtype=torch.uint8, device="cuda")
    bnd.as_accept_lm_head_sampled(vs.plan, hidden.cuda().contiguous(), weight.cuda().contiguous(), vs.draft_tokens, vs.draft_probs,
                                  vs.temperature, vs.u, vs.w, None, scratch, vs.accept_len, vs.out_tokens)
    torch.cuda.synchronize()
    assert bnd.as_plan_check(vs.plan) == 0
    in_band, total, exact = _check_sampled(bnd, A, vs, band=SAMPLED_BAND)
    assert in_band <= 1, (in_band, total)
    assert exact >= A.batch - 1, exact


def test_sampled_acceptance_from_hidden_states_with_uniforms_drawn_in_the_kernels(bnd):
    """rng_state instead of u / w: the decisions are the ones of the passed-in path fed with the oracle's Philox uniforms."""
    A, hidden, weight = _setup_sampled(31, [64] * 12, [5] * 12, 256, 3000, 0.8, True)
    seed, step = 0x9E3779B97F4A7C15, 7
    u, w_req = oracle.philox_uniforms(seed, step, A.draft_lens)
    cu_q, _ = cu(A.draft_lens)
    w = np.zeros(A.total_q, dtype=np.float32)               # the passed-in path reads w at row a_i: the same draw for every row
    for i in range(A.batch):
        w[cu_q[i]:cu_q[i + 1]] = w_req[i]
    A.u, A.w = u, w
    vs = bnd.VerifyStep(A)
    vs.plan_step()
    scratch = torch.empty(bnd.as_accept_lm_head_scratch_bytes(vs.plan, 256, 3000), dtype=torch.uint8, device="cuda")
    to_i64 = lambda x: x - (1 << 64) if x >= (1 << 63) else x
    state = torch.tensor([to_i64(seed), to_i64(step)], dtype=torch.int64, device="cuda")
    h, wt = hidden.cuda().contiguous(), weight.cuda().contiguous()
    bnd.as_accept_lm_head_sampled(vs.plan, h, wt, vs.draft_tokens, vs.draft_probs, vs.temperature, None, None, state, scratch,
                                  vs.accept_len, vs.out_tokens)
    a1, t1 = vs.accept_len.clone(), vs.out_tokens.clone()
    bnd.as_accept_lm_head_sampled(vs.plan, h, wt, vs.draft_tokens, vs.draft_probs, vs.temperature, vs.u, vs.w, None, scratch,
                                  vs.accept_len, vs.out_tokens)
    torch.cuda.synchronize()
    assert bnd.as_plan_check(vs.plan) == 0
    assert torch.equal(a1, vs.accept_len) and torch.equal(t1, vs.out_tokens)
