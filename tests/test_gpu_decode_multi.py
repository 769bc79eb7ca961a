"""GPU parity of seer_sparse_decode_multi / seer_dense_decode_multi (q_len query tokens per
sequence, causal among them) against the fp64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_08889_b200 import binding, synth
from util import bits, check_attention, to_paged, ref_sparse_multi, bf16_ulp

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", params=["mma.sync", "tcgen05"])
def ctx(request):
    """Every test of this file runs twice: units of 17 to 64 rows take the rows-on-M kernel, which exists as an
    mma.sync variant and as a tcgen05 variant (S, P, O and the queries in tensor memory); a context created with
    SEER_DECODE_WIDE_VARIANT=8 or 16 takes that one at every size (unset: tcgen05 up to 48 rows).  Up to 16 rows
    both runs take the same kernels."""
    import os
    old = os.environ.get("SEER_DECODE_WIDE_VARIANT")
    os.environ["SEER_DECODE_WIDE_VARIANT"] = "16" if request.param == "tcgen05" else "8"
    try:
        c = binding.Context(0)
    finally:
        if old is None:
            del os.environ["SEER_DECODE_WIDE_VARIANT"]
        else:
            os.environ["SEER_DECODE_WIDE_VARIANT"] = old
    yield c
    c.close()


def _make(B, T, Hq, Hkv, S, seed, name=""):
    q = synth.normal_bf16((B, T, Hq, 128), seed, name + "q", DEV)
    k = synth.normal_bf16((B, Hkv, S, 128), seed, name + "k", DEV)
    v = synth.normal_bf16((B, Hkv, S, 128), seed, name + "v", DEV)
    return q, k, v


def _run(ctx, q, k, v, lens, idx, cnt, b, scale, dense=False, page_table=None, page_size=0, max_seq_len=None):
    B, T, Hq, d = q.shape
    Hkv = k.shape[1]
    shape = binding.make_shape(B, Hq, Hkv, d, b, scale)
    lens_t = torch.as_tensor(np.asarray(lens, np.int32), device=DEV)
    kv = binding.make_kv(k, v, lens_t, max_seq_len=max_seq_len, page_table=page_table, page_size=page_size)
    out = torch.full((B, T, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, T, Hq), float("nan"), dtype=torch.float32, device=DEV)
    if dense:
        ctx.seer_dense_decode_multi(shape, kv, q, T, out, lse)
    else:
        idx_t = torch.as_tensor(idx, device=DEV).contiguous()
        cnt_t = None if cnt is None else torch.as_tensor(cnt, device=DEV).contiguous()
        ctx.seer_sparse_decode_multi(shape, kv, q, T, idx_t, cnt_t, idx.shape[2], out, lse)
    torch.cuda.synchronize()
    return out, lse


def _all_blocks(lens, Hkv, b):
    n = [-(-int(L) // b) for L in lens]
    idx = np.full((len(lens), Hkv, max(max(n), 1)), -1, np.int32)
    cnt = np.zeros((len(lens), Hkv), np.int32)
    for i, x in enumerate(n):
        idx[i, :, :x] = np.arange(x)
        cnt[i] = x
    return idx, cnt


# (Hq, Hkv, q_len): rows on the MMA N side and launches per call
#   (32,8,2): 8 rows, one N-tile      (40,8,3): 15 rows, two N-tiles     (64,8,2): 16 rows
#   (8,8,8): 8 rows   (16,8,8): 16 rows   (40,8,1): plain decode
# more than 16 rows take the variant with the rows on the MMA's M side, one launch for up to 64 rows:
#   (40,8,8): 40 rows   (64,8,8): 64 rows   (6,2,6): 18 rows   (56,8,8): 56 rows   (40,8,4): 20 rows
@pytest.mark.parametrize("Hq,Hkv,T", [(32, 8, 2), (40, 8, 3), (64, 8, 2), (40, 8, 8), (8, 8, 8), (16, 8, 8),
                                      (40, 8, 1), (6, 2, 5), (64, 8, 8), (6, 2, 6), (56, 8, 8), (40, 8, 4)])
def test_sparse_multi_ragged_lengths_and_boundaries(ctx, Hq, Hkv, T):
    B, S, b = 6, 1536, 64
    # 1536: full blocks; 1025: the last block holds one token, the others' own tokens sit in the block before;
    # 1027 / 517: tokens straddle a block (and tile) boundary for larger T; 70; 3: shorter than q_len for T > 3
    lens = np.array([1536, 1025, 1027, 517, 70, 3], np.int32)
    q, k, v = _make(B, T, Hq, Hkv, S, 700 + Hq + T)
    n = [-(-int(L) // b) for L in lens]
    keep = [max(1, x // 2) for x in n]
    idx, cnt = synth.random_block_lists(lens, Hkv, b, keep, max(keep) + 2, 700 + T, shuffle=True)
    ref = ref_sparse_multi(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.09)
    out, lse = _run(ctx, q, k, v, lens, idx, cnt, b, 0.09)
    check_attention(out, lse, *ref, what=f"multi Hq={Hq} T={T}")
    assert ctx.device_status() == binding.SEER_OK


@pytest.mark.parametrize("Hq,Hkv,T,b", [(40, 8, 3, 64), (32, 8, 4, 128), (64, 8, 4, 64)])
def test_dense_multi_equals_oracle_with_every_block_listed(ctx, Hq, Hkv, T, b):
    B, S = 4, 2048
    lens = np.array([2048, 1000, 65, 2], np.int32)
    q, k, v = _make(B, T, Hq, Hkv, S, 800 + T)
    idx, cnt = _all_blocks(lens, Hkv, b)
    ref = ref_sparse_multi(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.09)
    out, lse = _run(ctx, q, k, v, lens, None, None, b, 0.09, dense=True)
    check_attention(out, lse, *ref, what="dense multi")
    outs, lses = _run(ctx, q, k, v, lens, idx, cnt, b, 0.09)
    check_attention(outs, lses, *ref, what="sparse multi, all blocks")
    assert ctx.device_status() == binding.SEER_OK


def test_multi_rows_that_see_nothing_are_zero(ctx):
    # only the last block is listed and it holds one token: the earlier query tokens see nothing
    B, T, Hq, Hkv, S, b = 2, 3, 40, 8, 256, 64
    lens = np.array([129, 193], np.int32)
    q, k, v = _make(B, T, Hq, Hkv, S, 810)
    idx = np.array([[[2]] * Hkv, [[3]] * Hkv], np.int32)
    ref_o, ref_l, ref_a = ref_sparse_multi(bits(q), bits(k), bits(v), lens, idx, None, b, 0.09)
    assert np.isneginf(ref_l[:, :2]).all() and np.isfinite(ref_l[:, 2]).all()
    out, lse = _run(ctx, q, k, v, lens, idx, None, b, 0.09)
    check_attention(out, lse, ref_o, ref_l, ref_a, what="unseen rows")
    assert (out[:, :2] == 0).all()


def test_multi_long_lists_split_over_ctas_and_paged(ctx):
    # enough tiles per unit that every unit is cut into pieces and merged by the combine
    B, T, Hq, Hkv, S, b = 2, 3, 40, 8, 16384, 64
    lens = np.array([16384, 12345], np.int32)
    q, k, v = _make(B, T, Hq, Hkv, S, 820)
    n = [-(-int(L) // b) for L in lens]
    keep = [x // 2 for x in n]
    idx, cnt = synth.random_block_lists(lens, Hkv, b, keep, max(keep), 820)
    ref = oracle.sparse_multi(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.0884)
    out, lse = _run(ctx, q, k, v, lens, idx, cnt, b, 0.0884)
    check_attention(out, lse, *ref, what="multi long", strict=True)
    kp, vp, table = to_paged(k, v, b, 820)
    outp, lsep = _run(ctx, q, kp, vp, lens, idx, cnt, b, 0.0884, page_table=table, page_size=b, max_seq_len=S)
    check_attention(outp, lsep, *ref, what="multi long paged", strict=True)
    assert ctx.device_status() == binding.SEER_OK


@pytest.mark.parametrize("Hq,T", [(40, 8), (64, 8), (56, 7)])
def test_multi_many_rows_long_lists_dense_and_paged(ctx, Hq, T):
    # 17 to 64 rows per unit in one launch (rows on the MMA's M side): long lists cut into pieces and combined,
    # the dense call, and the same cache behind a page table, at the bound stated for long contexts
    B, Hkv, S, b = 2, 8, 16384, 64
    lens = np.array([16384, 12345], np.int32)
    q, k, v = _make(B, T, Hq, Hkv, S, 870 + T)
    n = [-(-int(L) // b) for L in lens]
    keep = [x // 2 for x in n]
    idx, cnt = synth.random_block_lists(lens, Hkv, b, keep, max(keep), 870 + T)
    ref = oracle.sparse_multi(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.0884)
    launches = ctx.launch_count()
    out, lse = _run(ctx, q, k, v, lens, idx, cnt, b, 0.0884)
    assert ctx.launch_count() - launches == 1
    check_attention(out, lse, *ref, what="many rows sparse", strict=True)
    kp, vp, table = to_paged(k, v, b, 870)
    outp, lsep = _run(ctx, q, kp, vp, lens, idx, cnt, b, 0.0884, page_table=table, page_size=b, max_seq_len=S)
    check_attention(outp, lsep, *ref, what="many rows paged", strict=True)
    full_idx, full_cnt = _all_blocks(lens, Hkv, b)
    refd = oracle.sparse_multi(bits(q), bits(k), bits(v), lens, full_idx, full_cnt, b, 0.0884)
    outd, lsed = _run(ctx, q, k, v, lens, None, None, b, 0.0884, dense=True)
    check_attention(outd, lsed, *refd, what="many rows dense", strict=True)
    assert ctx.device_status() == binding.SEER_OK


def test_multi_one_token_is_bitwise_the_single_token_call(ctx):
    B, Hq, Hkv, S, b = 3, 40, 8, 4096, 64
    lens = np.array([4096, 3000, 100], np.int32)
    q, k, v = _make(B, 1, Hq, Hkv, S, 830)
    idx, cnt = synth.random_block_lists(lens, Hkv, b, [20, 15, 2], 20, 830)
    out, lse = _run(ctx, q, k, v, lens, idx, cnt, b, 0.0884)
    shape = binding.make_shape(B, Hq, Hkv, 128, b, 0.0884)
    lens_t = torch.as_tensor(lens, device=DEV)
    kv = binding.make_kv(k, v, lens_t)
    out1 = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device=DEV)
    lse1 = torch.empty((B, Hq), dtype=torch.float32, device=DEV)
    ctx.seer_sparse_decode(shape, kv, q[:, 0].contiguous(), torch.as_tensor(idx, device=DEV),
                           torch.as_tensor(cnt, device=DEV), 20, out1, lse1)
    torch.cuda.synchronize()
    assert torch.equal(out[:, 0], out1) and torch.equal(lse[:, 0], lse1)


def test_multi_rejects_unsupported_q_len(ctx):
    B, Hq, Hkv, S, b = 1, 8, 8, 64, 64
    q, k, v = _make(B, 1, Hq, Hkv, S, 840)
    shape = binding.make_shape(B, Hq, Hkv, 128, b, 0.1)
    kv = binding.make_kv(k, v, torch.tensor([64], dtype=torch.int32, device=DEV))
    out = torch.empty_like(q)
    for bad in (0, 9):
        with pytest.raises(binding.SeerError):
            ctx.seer_dense_decode_multi(shape, kv, q, bad, out)


# ---- the gate for several query tokens -------------------------------------------------------------

THETA = 1.0e6


@pytest.mark.parametrize("g,T,b,dg", [(5, 3, 64, 128), (4, 8, 64, 64), (8, 2, 128, 128), (1, 5, 64, 256)])
def test_gate_multi_scores_and_selection(ctx, g, T, b, dg):
    B, Hkv, d = 4, 2, 128
    Hq = g * Hkv
    nbmax = 700
    # full; the T tokens straddle two blocks; exactly at a block end; shorter than T tokens
    lens = np.array([nbmax * b, 333 * b + 2, 100 * b, 3], np.int32)
    qn = synth.normal_bf16((B, T, Hq, d), 60 + T, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, g * d), 60 + T, "wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nbmax, dg), 60 + T, "kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nbmax)
    lens_t = torch.as_tensor(lens, device=DEV)
    max_sel = 70
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nbmax), dtype=torch.float32, device=DEV)
    ctx.seer_gate_select_multi(shape, gate, lens_t, qn, None, T, max_sel * b, idx, cnt, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    want_sc = oracle.scores_multi(bits(qn), bits(wq), bits(kc), lens, b, THETA)
    got_sc = sc.cpu().numpy()
    for i in range(B):
        jf = max(0, int(lens[i]) - T) // b
        if jf:
            assert np.abs(got_sc[i, :, :jf] - want_sc[i, :, :jf]).max() <= 1e-3
    # the selection is exact on the scores the GPU produced, for several budgets
    for budget in (max_sel * b, 3 * b, b, 0):
        ctx.seer_gate_select_multi(shape, gate, lens_t, qn, None, T, budget, idx, cnt, max_sel)
        torch.cuda.synchronize()
        want_idx, want_cnt = oracle.select_multi(got_sc, lens, b, budget, T, max_sel)
        assert np.array_equal(cnt.cpu().numpy(), want_cnt), budget
        assert np.array_equal(idx.cpu().numpy(), want_idx), budget
    # selection only, on given scores
    ctx.seer_gate_select_multi(shape, binding.make_gate(dg, THETA, None, None, None, nbmax), lens_t, None, sc, T, 20 * b,
                               idx, cnt, max_sel)
    torch.cuda.synchronize()
    want_idx, want_cnt = oracle.select_multi(got_sc, lens, b, 20 * b, T, max_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)
    assert ctx.device_status() == binding.SEER_OK


@pytest.mark.parametrize("g,T,dg", [(5, 3, 128), (4, 8, 64)])
def test_gate_multi_more_keys_than_one_cluster_holds(ctx, g, T, dg):
    # more than 8192 compressed keys per unit: the projection kernel makes one gate query per token,
    # the score kernel keeps per key the largest of the tokens' scores, the last slice selects
    B, Hkv, d, b = 2, 2, 128, 64
    Hq = g * Hkv
    nbmax = 9000
    lens = np.array([nbmax * b - 1, 8300 * b + 2], np.int32)     # the T tokens straddle two blocks in both
    qn = synth.normal_bf16((B, T, Hq, d), 90 + T, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, g * d), 90 + T, "wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nbmax, dg), 90 + T, "kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nbmax)
    lens_t = torch.as_tensor(lens, device=DEV)
    max_sel = 300
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nbmax), dtype=torch.float32, device=DEV)
    ctx.seer_gate_select_multi(shape, gate, lens_t, qn, None, T, max_sel * b, idx, cnt, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    want_sc = oracle.scores_multi(bits(qn), bits(wq), bits(kc), lens, b, THETA)
    got_sc = sc.cpu().numpy()
    for i in range(B):
        jf = max(0, int(lens[i]) - T) // b
        assert np.abs(got_sc[i, :, :jf] - want_sc[i, :, :jf]).max() <= 1e-3
    for budget in (max_sel * b, 17 * b):
        ctx.seer_gate_select_multi(shape, gate, lens_t, qn, None, T, budget, idx, cnt, max_sel)
        torch.cuda.synchronize()
        want_idx, want_cnt = oracle.select_multi(got_sc, lens, b, budget, T, max_sel)
        assert np.array_equal(cnt.cpu().numpy(), want_cnt), budget
        assert np.array_equal(idx.cpu().numpy(), want_idx), budget
    assert ctx.device_status() == binding.SEER_OK


@pytest.mark.parametrize("nbmax,tau,T", [(700, 2e-3, 3), (9000, 1.5e-4, 4)])
def test_gate_multi_threshold_method(ctx, nbmax, tau, T):
    # the threshold method with several query tokens, through both scoring paths: scores against the oracle,
    # the selection against the oracle's rule on the GPU's own scores (only blocks whose probability is
    # within rounding of tau may fall on either side)
    B, Hkv, g, d, dg, b = 2, 2, 4, 128, 128, 64
    Hq = g * Hkv
    max_sel = nbmax // 2
    lens = np.array([nbmax * b - 1, (nbmax // 2) * b + 2], np.int32)
    qn = synth.normal_bf16((B, T, Hq, d), 77, "thr:qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, g * d), 77, "thr:wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nbmax, dg), 77, "thr:kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nbmax)
    lens_t = torch.as_tensor(lens, device=DEV)
    idx = torch.full((B, Hkv, max_sel), 77, dtype=torch.int32, device=DEV)
    cnt = torch.full((B, Hkv), 77, dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nbmax), dtype=torch.float32, device=DEV)
    ctx.seer_gate_select_threshold_multi(shape, gate, lens_t, qn, None, T, tau, idx, cnt, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    want_sc = oracle.scores_multi(bits(qn), bits(wq), bits(kc), lens, b, THETA)
    got_sc = sc.cpu().numpy()
    for i in range(B):
        jf = max(0, int(lens[i]) - T) // b
        assert np.abs(got_sc[i, :, :jf] - want_sc[i, :, :jf]).max() <= 1e-3
    want_idx, want_cnt, probs = oracle.select_threshold_multi(got_sc, lens, b, tau, T, max_sel)
    idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
    for i in range(B):
        L = int(lens[i])
        n, jf = -(-L // b), max(0, L - T) // b
        for h in range(Hkv):
            got = set(idx[i, h, :cnt[i, h]].tolist())
            want = set(want_idx[i, h, :want_cnt[i, h]].tolist())
            assert set(range(jf, n)) <= got and list(idx[i, h, :cnt[i, h]]) == sorted(got)
            assert np.all(idx[i, h, cnt[i, h]:] == -1)
            for j in got ^ want:
                assert abs(probs[i, h, j] - tau) <= 1e-5 * tau + 1e-9, (i, h, j, probs[i, h, j])
            assert n - jf < len(got) < n                     # the threshold cut somewhere inside
    assert ctx.device_status() == binding.SEER_OK


def test_gate_multi_with_one_token_is_bitwise_the_single_token_gate(ctx):
    B, Hq, Hkv, d, dg, b, nbmax = 3, 40, 8, 128, 128, 64, 2048
    lens = np.array([nbmax * b, 1000 * b + 17, 64], np.int32)
    qn = synth.normal_bf16((B, 1, Hq, d), 70, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, 5 * d), 70, "wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nbmax, dg), 70, "kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nbmax)
    lens_t = torch.as_tensor(lens, device=DEV)
    res = []
    for multi in (False, True):
        idx = torch.zeros((B, Hkv, 205), dtype=torch.int32, device=DEV)
        cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
        sc = torch.zeros((B, Hkv, nbmax), dtype=torch.float32, device=DEV)
        if multi:
            ctx.seer_gate_select_multi(shape, gate, lens_t, qn, None, 1, 205 * b, idx, cnt, 205, scores_out=sc)
        else:
            ctx.seer_gate_select(shape, gate, lens_t, qn[:, 0].contiguous(), None, 205 * b, idx, cnt, 205, scores_out=sc)
        torch.cuda.synchronize()
        res.append((idx, cnt, sc))
    for a, c in zip(res[0], res[1]):
        assert torch.equal(a, c)


def test_multi_token_step_gate_then_decode(ctx):
    # three query tokens per sequence through the gate and the decode kernel, 14B head counts
    B, T, Hq, Hkv, d, dg, b, L = 2, 3, 40, 8, 128, 128, 64, 16384
    nb = L // b
    lens = np.array([L, L - 1000], np.int32)
    q, k, v = _make(B, T, Hq, Hkv, L, 90)
    qn = synth.normal_bf16((B, T, Hq, d), 90, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, 5 * d), 90, "wq", DEV, std=0.02)
    wk = synth.normal_bf16((Hkv, dg, 3 * d), 90, "wk", DEV, std=0.02)
    kc = torch.zeros((B, Hkv, nb, dg), dtype=torch.bfloat16, device=DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.0884)
    gate = binding.make_gate(dg, THETA, wq, wk, kc, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    ctx.seer_kcomp_append(shape, gate, lens_t, k, first_block=0, num_blocks=nb)
    max_sel = 26                                                  # s = 0.9
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nb), dtype=torch.float32, device=DEV)
    ctx.seer_gate_select_multi(shape, gate, lens_t, qn, None, T, max_sel * b, idx, cnt, max_sel, scores_out=sc)
    kv = binding.make_kv(k, v, lens_t)
    out = torch.full((B, T, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, T, Hq), float("nan"), dtype=torch.float32, device=DEV)
    ctx.seer_sparse_decode_multi(shape, kv, q, T, idx, cnt, max_sel, out, lse)
    torch.cuda.synchronize()
    want_idx, want_cnt = oracle.select_multi(sc.cpu().numpy(), lens, b, max_sel * b, T, max_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)
    ref = oracle.sparse_multi(bits(q), bits(k), bits(v), lens, want_idx, want_cnt, b, 0.0884)
    check_attention(out, lse, *ref, what="multi step", strict=True)
    # every query token sees at least itself: its own block is in the list
    assert np.isfinite(ref[1]).all()
    assert ctx.device_status() == binding.SEER_OK


def test_multi_token_step_call_appends_the_block_that_filled_among_the_new_tokens(ctx):
    # q_len = 4 tokens have just been appended; lengths: a block boundary crossed two tokens ago
    # (L % b = 2 < 4: block L/b - 1 is written), exactly at a boundary, and no boundary crossed
    B, T, Hq, Hkv, d, dg, b, S = 3, 4, 32, 8, 128, 128, 64, 4096
    nb = S // b
    lens = np.array([40 * b + 2, 64 * b, 50 * b + 9], np.int32)
    q, k, v = _make(B, T, Hq, Hkv, S, 95)
    qn = synth.normal_bf16((B, T, Hq, d), 95, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, 4 * d), 95, "wq", DEV, std=0.02)
    wk = synth.normal_bf16((Hkv, dg, 3 * d), 95, "wk", DEV, std=0.02)
    kc = torch.zeros((B, Hkv, nb, dg), dtype=torch.bfloat16, device=DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.0884)
    gate = binding.make_gate(dg, THETA, wq, wk, kc, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    # the cache as it stood before these T tokens: every block complete by then
    before = torch.as_tensor(lens - T, device=DEV)
    ctx.seer_kcomp_append(shape, gate, before, k, first_block=0, num_blocks=nb)
    torch.cuda.synchronize()
    kc_before = kc.clone()
    kv = binding.make_kv(k, v, lens_t)
    max_sel = 8
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    out = torch.full((B, T, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, T, Hq), float("nan"), dtype=torch.float32, device=DEV)
    ctx.seer_decode_step_multi(shape, kv, gate, q, qn, T, k, max_sel * b, idx, cnt, max_sel, out, lse)
    torch.cuda.synchronize()
    # compressed keys: sequences 0 and 1 got the entry of the block that filled, sequence 2 nothing
    _, want = oracle.kcomp(bits(k), bits(wk), b, 0, nb, nb, THETA)
    got = synth.bits_to_bf16(bits(kc)).to(torch.float64).numpy()
    for i, j in ((0, 39), (1, 63)):
        assert (kc_before[i, :, j] == 0).all()
        tol = bf16_ulp(want[i, :, j]) + 1e-5 * np.abs(want).max()
        assert (np.abs(got[i, :, j] - want[i, :, j]) <= tol).all()
    changed = (kc != kc_before).any(dim=3).cpu().numpy()
    assert changed[0, :, 39].all() and changed[1, :, 63].all() and changed.sum() == 2 * Hkv
    # the lists and the attention are what the separate calls give on the updated cache
    sc = torch.zeros((B, Hkv, nb), dtype=torch.float32, device=DEV)
    idx2, cnt2 = torch.zeros_like(idx), torch.zeros_like(cnt)
    ctx.seer_gate_select_multi(shape, gate, lens_t, qn, None, T, max_sel * b, idx2, cnt2, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    assert torch.equal(idx, idx2) and torch.equal(cnt, cnt2)
    want_idx, want_cnt = oracle.select_multi(sc.cpu().numpy(), lens, b, max_sel * b, T, max_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)
    ref = ref_sparse_multi(bits(q), bits(k), bits(v), lens, want_idx, want_cnt, b, 0.0884)
    check_attention(out, lse, *ref, what="multi step call")
    assert ctx.device_status() == binding.SEER_OK
