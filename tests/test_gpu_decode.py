"""GPU parity of seer_sparse_decode / seer_dense_decode against the fp64 oracle, element by
element on seeded inputs, called through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_08889_b200 import binding, synth
from util import bits, check_attention, make_qkv, to_paged, ref_sparse, ref_dense

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def _run_sparse(ctx, q, k, v, lens, idx, cnt, b, scale, page_table=None, page_size=0, max_seq_len=None,
                use_cnt=True):
    B, Hq, d = q.shape
    Hkv = k.shape[1]
    shape = binding.make_shape(B, Hq, Hkv, d, b, scale)
    lens_t = torch.as_tensor(np.asarray(lens, np.int32), device=DEV)
    kv = binding.make_kv(k, v, lens_t, max_seq_len=max_seq_len, page_table=page_table, page_size=page_size)
    idx_t = torch.as_tensor(idx, device=DEV).contiguous()
    cnt_t = torch.as_tensor(cnt, device=DEV).contiguous() if (use_cnt and cnt is not None) else None
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
    ctx.seer_sparse_decode(shape, kv, q, idx_t, cnt_t, idx.shape[2], out, lse)
    torch.cuda.synchronize()
    return out, lse


def _run_dense(ctx, q, k, v, lens, b, scale, page_table=None, page_size=0, max_seq_len=None):
    B, Hq, d = q.shape
    Hkv = k.shape[1]
    shape = binding.make_shape(B, Hq, Hkv, d, b, scale)
    lens_t = torch.as_tensor(np.asarray(lens, np.int32), device=DEV)
    kv = binding.make_kv(k, v, lens_t, max_seq_len=max_seq_len, page_table=page_table, page_size=page_size)
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
    ctx.seer_dense_decode(shape, kv, q, out, lse)
    torch.cuda.synchronize()
    return out, lse


def test_tiny_workload_every_element(ctx):
    w = synth.workload(0)
    lens = w.lengths()
    q, k, v = make_qkv(w.batch, w.num_q_heads, w.num_kv_heads, w.seq_len, w.head_dim, synth.BASE_SEED, DEV, w.name)
    idx, cnt = synth.random_block_lists(lens, w.num_kv_heads, w.block_size, 8, 8, synth.BASE_SEED, w.name)
    assert idx[0, 0, -1] == 63 and cnt[0, 0] == 8
    out, lse = _run_sparse(ctx, q, k, v, lens, idx, cnt, w.block_size, w.sm_scale)
    ref_o, ref_l = oracle.sparse(bits(q), bits(k), bits(v), lens, idx, cnt, w.block_size, w.sm_scale)
    check_attention(out, lse, ref_o, ref_l, what="tiny", strict=True)
    assert ctx.device_status() == binding.SEER_OK


@pytest.mark.parametrize("g,Hkv,b,token_major", [(4, 2, 64, False), (5, 2, 64, True), (8, 1, 128, False),
                                                 (1, 3, 128, True), (2, 2, 64, False)])
def test_sparse_ragged_shuffled_lists(ctx, g, Hkv, b, token_major):
    B, d, S = 3, 128, 2048
    Hq = g * Hkv
    lens = np.array([2048, 1000, 517], np.int32)          # 517: partial tail; 1000 likewise
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 100 + g, DEV, token_major=token_major)
    n = [-(-int(L) // b) for L in lens]
    keep = [max(1, x // 3) for x in n]
    max_sel = max(keep) + 3
    idx, cnt = synth.random_block_lists(lens, Hkv, b, keep, max_sel, 100 + g, shuffle=True)
    ref = ref_sparse(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.09)
    out, lse = _run_sparse(ctx, q, k, v, lens, idx, cnt, b, 0.09)
    check_attention(out, lse, *ref, what=f"g={g}")
    # same lists without counts: the -1 padding is skipped
    out2, lse2 = _run_sparse(ctx, q, k, v, lens, idx, cnt, b, 0.09, use_cnt=False)
    check_attention(out2, lse2, *ref, what=f"g={g} no-cnt")
    assert ctx.device_status() == binding.SEER_OK


def test_rows_past_the_length_are_never_used(ctx):
    # the cache rows beyond L_i hold NaN and huge values: the result must not change
    B, Hq, Hkv, d, b, S = 2, 8, 2, 128, 64, 512
    lens = np.array([300, 65], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 7, DEV)
    for i, L in enumerate(lens):
        k[i, :, L:] = float("nan")
        v[i, :, L:] = float("nan")
    k[0, :, 310] = 1e30
    idx, cnt = synth.random_block_lists(lens, Hkv, b, [3, 2], 4, 7)
    kh, vh = torch.nan_to_num(k, nan=0.0).cpu(), torch.nan_to_num(v, nan=0.0).cpu()
    ref = ref_sparse(bits(q), bits(kh), bits(vh), lens, idx, cnt, b, 0.1)
    out, lse = _run_sparse(ctx, q, k, v, lens, idx, cnt, b, 0.1)
    check_attention(out, lse, *ref, what="nan tail sparse")
    refd = ref_dense(bits(q), bits(kh), bits(vh), lens, 0.1)
    outd, lsed = _run_dense(ctx, q, k, v, lens, b, 0.1)
    check_attention(outd, lsed, *refd, what="nan tail dense")


@pytest.mark.parametrize("b", [64, 128])
def test_dense_ragged_lengths(ctx, b):
    B, Hq, Hkv, d, S = 6, 10, 2, 128, 1536
    lens = np.array([1, 64, 65, 1536, 0, 777], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 33, DEV)
    ref = ref_dense(bits(q), bits(k), bits(v), lens, 0.0884)
    out, lse = _run_dense(ctx, q, k, v, lens, b, 0.0884)
    check_attention(out, lse, *ref, what="dense ragged")
    assert torch.all(out[4] == 0) and torch.all(torch.isneginf(lse[4]))


def test_full_selection_matches_dense_kernel_and_oracle(ctx):
    B, Hq, Hkv, d, b, S = 2, 8, 2, 128, 64, 4096
    lens = np.array([4096, 2500], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 44, DEV)
    n = [-(-int(L) // b) for L in lens]
    idx = np.full((B, Hkv, 64), -1, np.int32)
    cnt = np.zeros((B, Hkv), np.int32)
    for i in range(B):
        idx[i, :, :n[i]] = np.arange(n[i])
        cnt[i] = n[i]
    ref = oracle.dense(bits(q), bits(k), bits(v), lens, 0.0884)
    out_s, lse_s = _run_sparse(ctx, q, k, v, lens, idx, cnt, b, 0.0884)
    out_d, lse_d = _run_dense(ctx, q, k, v, lens, b, 0.0884)
    check_attention(out_s, lse_s, *ref, what="100% selection", strict=True)
    check_attention(out_d, lse_d, *ref, what="dense", strict=True)


def test_one_long_unit_is_split_over_many_ctas(ctx):
    # a single (sequence, KV head) pair: every CTA holds a piece, one combine of ~300 partials
    B, Hq, Hkv, d, b, S = 1, 4, 1, 128, 64, 65536
    lens = np.array([S - 11], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 55, DEV)
    ref = oracle.dense(bits(q), bits(k), bits(v), lens, 0.0884)
    out, lse = _run_dense(ctx, q, k, v, lens, b, 0.0884)
    check_attention(out, lse, *ref, what="long dense", strict=True)
    idx, cnt = synth.random_block_lists(lens, Hkv, b, 700, 700, 55)
    ref = oracle.sparse(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.0884)
    for _ in range(3):                                    # tickets must be reusable launch after launch
        out, lse = _run_sparse(ctx, q, k, v, lens, idx, cnt, b, 0.0884)
        check_attention(out, lse, *ref, what="long sparse", strict=True)


@pytest.mark.parametrize("b,page_size", [(64, 64), (128, 128), (64, 256)])
def test_paged_cache(ctx, b, page_size):
    B, Hq, Hkv, d, S = 3, 8, 2, 128, 2048
    lens = np.array([2048, 1300, 70], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 66, DEV)
    kp, vp, table = to_paged(k, v, page_size, 66)
    n = [-(-int(L) // b) for L in lens]
    idx, cnt = synth.random_block_lists(lens, Hkv, b, [max(1, x // 2) for x in n], max(n), 66, shuffle=True)
    ref = ref_sparse(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.0884)
    out, lse = _run_sparse(ctx, q, kp, vp, lens, idx, cnt, b, 0.0884, page_table=table, page_size=page_size,
                           max_seq_len=S)
    check_attention(out, lse, *ref, what="paged sparse")
    refd = ref_dense(bits(q), bits(k), bits(v), lens, 0.0884)
    outd, lsed = _run_dense(ctx, q, kp, vp, lens, b, 0.0884, page_table=table, page_size=page_size, max_seq_len=S)
    check_attention(outd, lsed, *refd, what="paged dense")
    assert ctx.device_status() == binding.SEER_OK


def test_bad_entries_are_skipped_and_flagged(ctx):
    B, Hq, Hkv, d, b, S = 1, 8, 2, 128, 64, 1024
    lens = np.array([1000], np.int32)                      # 16 blocks
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 77, DEV)
    idx = np.array([[[3, 16, 9, -1, 15, 400], [-1, -1, 2, 15, 1 << 30, -5]]], np.int32)
    cnt = np.array([[6, 6]], np.int32)
    ref = ref_sparse(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.1)      # oracle ignores them
    out, lse = _run_sparse(ctx, q, k, v, lens, idx, cnt, b, 0.1)
    check_attention(out, lse, *ref, what="bad entries")
    assert ctx.device_status() == binding.SEER_ERR_BAD_INDEX
    assert ctx.device_status() == binding.SEER_OK          # reading clears the flag
    # a page id outside the pool is skipped and flagged too
    kp, vp, table = to_paged(k, v, 64, 77)
    table2 = table.clone()
    table2[0, 3] = kp.shape[0] + 5
    good = np.array([[[3, 9, 15, -1, -1, -1], [2, 15, -1, -1, -1, -1]]], np.int32)
    without3 = np.array([[[9, 15, -1, -1, -1, -1], [2, 15, -1, -1, -1, -1]]], np.int32)
    ref = ref_sparse(bits(q), bits(k), bits(v), lens, without3, None, b, 0.1)
    out, lse = _run_sparse(ctx, q, kp, vp, lens, good, None, b, 0.1, page_table=table2, page_size=64,
                           max_seq_len=S, use_cnt=False)
    check_attention(out, lse, *ref, what="bad page")
    assert ctx.device_status() == binding.SEER_ERR_BAD_INDEX


def test_empty_lists_give_zero_and_minus_inf(ctx):
    B, Hq, Hkv, d, b, S = 2, 8, 2, 128, 64, 256
    lens = np.array([256, 200], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 88, DEV)
    idx = np.full((B, Hkv, 4), -1, np.int32)
    idx[1, 1, :2] = [0, 3]
    cnt = np.zeros((B, Hkv), np.int32)
    cnt[1, 1] = 2
    cnt[0, 1] = 3                                          # counted but all padding
    ref = ref_sparse(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.1)
    out, lse = _run_sparse(ctx, q, k, v, lens, idx, cnt, b, 0.1)
    check_attention(out, lse, *ref, what="empty")
    assert torch.all(out[0] == 0) and torch.all(torch.isneginf(lse[0]))


def test_host_side_argument_checks(ctx):
    B, Hq, Hkv, d, S = 1, 8, 2, 128, 256
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 99, DEV)
    lens_t = torch.tensor([256], dtype=torch.int32, device=DEV)
    out = torch.empty_like(q)
    kv = binding.make_kv(k, v, lens_t)
    for bad_shape, status in [
        (binding.make_shape(B, Hq, Hkv, 64, 64, 0.1), binding.SEER_ERR_UNSUPPORTED),
        (binding.make_shape(B, Hq, Hkv, d, 48, 0.1), binding.SEER_ERR_UNSUPPORTED),
        (binding.make_shape(B, 9, 2, d, 64, 0.1), binding.SEER_ERR_INVALID_ARG),
        (binding.make_shape(B, 32, 2, d, 64, 0.1), binding.SEER_ERR_UNSUPPORTED),
        (binding.make_shape(0, Hq, Hkv, d, 64, 0.1), binding.SEER_ERR_INVALID_ARG),
    ]:
        with pytest.raises(binding.SeerError) as e:
            ctx.seer_dense_decode(bad_shape, kv, q, out)
        assert e.value.status == status
    shape = binding.make_shape(B, Hq, Hkv, d, 64, 0.1)
    with pytest.raises(binding.SeerError) as e:
        ctx.seer_sparse_decode(shape, kv, q, None, None, 4, out)
    assert e.value.status == binding.SEER_ERR_INVALID_ARG
    kv_bad = binding.make_kv(k[:, :, :, 1:], v[:, :, :, 1:], lens_t)      # misaligned base
    with pytest.raises(binding.SeerError) as e:
        ctx.seer_dense_decode(shape, kv_bad, q, out)
    assert e.value.status == binding.SEER_ERR_INVALID_ARG
    small = binding.Context(0, workspace_bytes=4096)
    with pytest.raises(binding.SeerError) as e:
        small.seer_dense_decode(shape, kv, q, out)
    assert e.value.status == binding.SEER_ERR_WORKSPACE
    small.close()


def test_result_does_not_depend_on_how_the_work_is_cut(ctx, monkeypatch):
    # the same launch with work stealing (default) and with a purely static split, on a case large
    # enough for stealing to happen: both within the parity bound of the oracle, and of each other
    B, Hq, Hkv, d, b, S = 4, 10, 2, 128, 64, 32768
    lens = np.array([S, S - 1000, S // 2 + 17, S - 64], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 123, DEV)
    n = [-(-int(L) // b) for L in lens]
    idx, cnt = synth.random_block_lists(lens, Hkv, b, [x // 2 for x in n], max(n) // 2 + 1, 123)
    ref = oracle.sparse(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.0884)
    out_dyn, lse_dyn = _run_sparse(ctx, q, k, v, lens, idx, cnt, b, 0.0884)
    check_attention(out_dyn, lse_dyn, *ref, what="stealing", strict=True)
    monkeypatch.setenv("SEER_DECODE_POOL_DIV", "0")            # read when a context is created
    static_ctx = binding.Context(0)
    try:
        out_st, lse_st = _run_sparse(static_ctx, q, k, v, lens, idx, cnt, b, 0.0884)
    finally:
        static_ctx.close()
    check_attention(out_st, lse_st, *ref, what="static", strict=True)
    assert (out_dyn.float() - out_st.float()).abs().max().item() <= 2e-3
    # launch after launch on the same context: counters and tickets re-arm themselves
    for _ in range(5):
        o2, l2 = _run_sparse(ctx, q, k, v, lens, idx, cnt, b, 0.0884)
        check_attention(o2, l2, *ref, what="repeat", strict=True)
    assert ctx.device_status() == binding.SEER_OK


def test_counts_rewritten_by_the_kernel_just_before(ctx):
    # The kernel launched just before the sparse decode (a selection on given scores) rewrites counts
    # and lists every time, with a budget that alternates, and nothing synchronises in between: the
    # decode kernel may begin its set-up under that kernel's tail, but every result must be the
    # oracle's for the lists of its own step.
    B, Hq, Hkv, d, b, nb = 2, 8, 4, 128, 64, 96
    S = nb * b
    lens = np.array([S, S - 3 * b - 11], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 77, DEV)
    r = synth.np_rng(77, "scores")
    sc = r.normal(size=(B, Hkv, nb)).astype(np.float32)
    sc_t = torch.as_tensor(sc, device=DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.0884)
    gate = binding.make_gate(128, 1.0e6, None, None, None, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    kv = binding.make_kv(k, v, lens_t)
    max_sel = 40
    budgets = [5 * b, 37 * b]
    want = []
    for bud in budgets:
        i_w, c_w = oracle.select(sc, lens, b, bud, max_sel)
        want.append((i_w, c_w, ref_sparse(bits(q), bits(k), bits(v), lens, i_w, c_w, b, 0.0884)))
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    steps = 24
    outs = [torch.zeros((B, Hq, d), dtype=torch.bfloat16, device=DEV) for _ in range(steps)]
    lses = [torch.zeros((B, Hq), dtype=torch.float32, device=DEV) for _ in range(steps)]
    torch.cuda.synchronize()
    for s in range(steps):
        ctx.seer_gate_select(shape, gate, lens_t, None, sc_t, budgets[s & 1], idx, cnt, max_sel)
        ctx.seer_sparse_decode(shape, kv, q, idx, cnt, max_sel, outs[s], lses[s])
    torch.cuda.synchronize()
    for s in range(steps):
        o_w, l_w, a_w = want[s & 1][2]
        check_attention(outs[s], lses[s], o_w, l_w, a_w, what=f"step {s}")
    assert np.array_equal(idx.cpu().numpy(), want[(steps - 1) & 1][0])
    assert np.array_equal(cnt.cpu().numpy(), want[(steps - 1) & 1][1])
    assert ctx.device_status() == binding.SEER_OK


def test_decode_refuses_a_stream_that_is_being_captured(ctx):
    # a decode launch carries per-call counters, so a graph captured from it could not be replayed:
    # the call must say so instead of enqueueing anything, and work again once the capture is over
    B, Hq, Hkv, d, b, S = 1, 4, 1, 128, 64, 1024
    lens = np.array([S], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 5, DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.0884)
    lens_t = torch.as_tensor(lens, device=DEV)      # (kept alive: the kv struct holds its address only)
    kv = binding.make_kv(k, v, lens_t)
    out = torch.zeros((B, Hq, d), dtype=torch.bfloat16, device=DEV)
    fill = torch.zeros(8, device=DEV)
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        graph.capture_begin()
        try:
            fill.add_(1.0)                         # (something to capture, so that the graph is not empty)
            with pytest.raises(binding.SeerError) as e:
                ctx.seer_dense_decode(shape, kv, q, out, stream=side)
            assert e.value.status == binding.SEER_ERR_UNSUPPORTED
        finally:
            graph.capture_end()
    torch.cuda.synchronize()
    ctx.seer_dense_decode(shape, kv, q, out)
    torch.cuda.synchronize()
    ref = ref_dense(bits(q), bits(k), bits(v), lens, 0.0884)
    check_attention(out, None, ref[0], None, ref[2], what="after the capture")
    assert ctx.device_status() == binding.SEER_OK
