"""Parity on the specified workloads at full size, in the launch configuration the benchmark
times (contiguous head-major caches, counts given, default context), through the C ABI.

The fp64 oracle checks every output of the sparse path (its cost scales with the selected
tokens only) and every output of the dense path where that stays within seconds; selection is
compared bit for bit on the fp32 scores the GPU used."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_08889_b200 import binding, synth
from util import bits, check_attention, to_paged, kc_tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SEED = synth.BASE_SEED


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def _kv(w, tag):
    shape = (w.batch, w.num_kv_heads, w.seq_len, w.head_dim)
    return (synth.normal_bf16(shape, SEED, tag + "k", DEV), synth.normal_bf16(shape, SEED, tag + "v", DEV))


def _select_on_scores(ctx, w, lens, scores, max_sel, budgets=None):
    """Top-k through seer_gate_select on given scores; per-sequence budgets via one call each when
    the kept count differs between sequences (ragged workload)."""
    B, Hkv, b = w.batch, w.num_kv_heads, w.block_size
    lens_t = torch.as_tensor(lens, device=DEV)
    idx = torch.full((B, Hkv, max_sel), -1, dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    gate = binding.make_gate(w.d_gate, w.rope_theta, None, None, None, scores.shape[2])
    if budgets is None:
        shape = binding.make_shape(B, w.num_q_heads, Hkv, w.head_dim, b, w.sm_scale)
        ctx.seer_gate_select(shape, gate, lens_t, None, scores, w.keep(lens[0] // b) * b, idx, cnt, max_sel)
    else:
        shape1 = binding.make_shape(1, w.num_q_heads, Hkv, w.head_dim, b, w.sm_scale)
        for i in range(B):
            ctx.seer_gate_select(shape1, gate, lens_t[i:i + 1], None, scores[i:i + 1], int(budgets[i]),
                                 idx[i:i + 1], cnt[i:i + 1], max_sel)
    torch.cuda.synchronize()
    return idx, cnt


def _decode_and_check(ctx, w, q, k, v, lens, idx, cnt, what, dense=False, page_table=None, page_size=0,
                      k_host=None, v_host=None):
    B, Hq, Hkv, d, b = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size
    shape = binding.make_shape(B, Hq, Hkv, d, b, w.sm_scale)
    lens_t = torch.as_tensor(lens, device=DEV)
    kv = binding.make_kv(k, v, lens_t, max_seq_len=w.seq_len, page_table=page_table, page_size=page_size)
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
    ctx.seer_sparse_decode(shape, kv, q, idx, cnt, idx.shape[2], out, lse)
    torch.cuda.synchronize()
    kh = bits(k) if k_host is None else k_host
    vh = bits(v) if v_host is None else v_host
    ref = oracle.sparse(bits(q), kh, vh, lens, idx.cpu().numpy(), cnt.cpu().numpy(), b, w.sm_scale)
    check_attention(out, lse, *ref, what=what + " sparse", strict=True)
    if dense:
        outd = torch.full_like(out, float("nan"))
        lsed = torch.full_like(lse, float("nan"))
        ctx.seer_dense_decode(shape, kv, q, outd, lsed)
        torch.cuda.synchronize()
        refd = oracle.dense(bits(q), kh, vh, lens, w.sm_scale)
        check_attention(outd, lsed, *refd, what=what + " dense", strict=True)
    assert ctx.device_status() == binding.SEER_OK
    return kh, vh


def test_qwen3_8b_shape_budget_4096(ctx):
    w = synth.workload(1)
    lens = w.lengths()
    nb = w.seq_len // w.block_size
    q = synth.normal_bf16((w.batch, w.num_q_heads, w.head_dim), SEED, w.name + "q", DEV)
    k, v = _kv(w, w.name)
    scores = synth.normal_f32((w.batch, w.num_kv_heads, nb), SEED, w.name + "scores", DEV)
    idx, cnt = _select_on_scores(ctx, w, lens, scores, 64)
    want_idx, want_cnt = oracle.select(scores.cpu().numpy(), lens, w.block_size, w.token_budget, 64)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)
    assert int(cnt[0, 0]) == 64 and int(idx[0, 0, 63]) == nb - 1
    kh, vh = _decode_and_check(ctx, w, q, k, v, lens, idx, cnt, "8b", dense=True)
    # the same cache behind a page table (page = block)
    kp, vp, table = to_paged(k, v, w.block_size, SEED)
    _decode_and_check(ctx, w, q, kp, vp, lens, idx, cnt, "8b paged", dense=True, page_table=table,
                      page_size=w.block_size, k_host=kh, v_host=vh)


def test_qwen3_14b_shape_gate_then_decode(ctx):
    w = synth.workload(2)
    lens = w.lengths()
    B, Hq, Hkv, d, b, L = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size, w.seq_len
    nb = L // b
    q = synth.normal_bf16((B, Hq, d), SEED, w.name + "q", DEV)
    qn = synth.normal_bf16((B, Hq, d), SEED, w.name + "qn", DEV)
    k, v = _kv(w, w.name)
    wq = synth.normal_bf16((Hkv, w.d_gate, w.group * d), SEED, w.name + "wq", DEV, std=w.gate_weight_std)
    wk = synth.normal_bf16((Hkv, w.d_gate, 3 * d), SEED, w.name + "wk", DEV, std=w.gate_weight_std)
    kc = torch.zeros((B, Hkv, nb, w.d_gate), dtype=torch.bfloat16, device=DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, w.sm_scale)
    gate = binding.make_gate(w.d_gate, w.rope_theta, wq, wk, kc, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    max_sel = w.token_budget // b
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nb), dtype=torch.float32, device=DEV)
    ctx.seer_kcomp_append(shape, gate, lens_t, k, first_block=0, num_blocks=nb)      # K_nope := K cache
    ctx.seer_gate_select(shape, gate, lens_t, qn, None, w.token_budget, idx, cnt, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    kh = bits(k)
    # stage 1: 1024 compressed keys per head, within one bf16 ulp
    _, kc_want = oracle.kcomp(kh, bits(wk), b, 0, nb, nb, w.rope_theta)
    got_kc = bits(kc)
    got = synth.bits_to_bf16(got_kc).to(torch.float64).numpy()
    tol = kc_tolerance(kc_want)
    assert (np.abs(got - kc_want) <= tol).all()
    # stage 2: scores on the GPU's compressed keys
    want_sc, _ = oracle.scores(bits(qn), bits(wq), got_kc, [nb - 1] * B, [L - 1] * B, w.rope_theta)
    got_sc = sc.cpu().numpy()
    assert np.abs(got_sc[:, :, :nb - 1] - want_sc[:, :, :nb - 1]).max() <= 1e-3
    # stage 3: the selection, exact on the GPU's scores
    want_idx, want_cnt = oracle.select(got_sc, lens, b, w.token_budget, max_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)
    # stage 4: attention over those lists
    _decode_and_check(ctx, w, q, k, v, lens, idx, cnt, "14b", dense=True, k_host=kh)


def test_qwen3_4b_shape_ragged_batch_block_128(ctx):
    w = synth.workload(3)
    lens = w.lengths()
    assert lens.min() >= 8192 and lens.max() <= 65536 and (lens % 128 == 0).all()
    B, Hkv, b = w.batch, w.num_kv_heads, w.block_size
    n = lens // b
    keep = np.array([w.keep(int(x)) for x in n])
    max_sel = int(keep.max())
    q = synth.normal_bf16((B, w.num_q_heads, w.head_dim), SEED, w.name + "q", DEV)
    k, v = _kv(w, w.name)
    scores = synth.normal_f32((B, Hkv, w.seq_len // b), SEED, w.name + "scores", DEV)
    idx, cnt = _select_on_scores(ctx, w, lens, scores, max_sel, budgets=keep * b)
    sc_h = scores.cpu().numpy()
    for i in range(B):
        wi, wc = oracle.select(sc_h[i:i + 1], lens[i:i + 1], b, int(keep[i] * b), max_sel)
        assert np.array_equal(idx[i:i + 1].cpu().numpy(), wi) and np.array_equal(cnt[i:i + 1].cpu().numpy(), wc)
    assert np.array_equal(cnt.cpu().numpy(), np.repeat(keep[:, None], Hkv, 1))
    kh, vh = _decode_and_check(ctx, w, q, k, v, lens, idx, cnt, "4b ragged", dense=True)
    kp, vp, table = to_paged(k, v, b, SEED)
    del k, v
    _decode_and_check(ctx, w, q, kp, vp, lens, idx, cnt, "4b ragged paged", page_table=table, page_size=b,
                      k_host=kh, v_host=vh)


@pytest.mark.parametrize("sparsity", [0.9, 0.5])
def test_qwen3_14b_long_context_sweep_point(ctx, sparsity):
    w = synth.workload(4)
    w.sparsity = sparsity
    lens = w.lengths()
    nb = w.seq_len // w.block_size
    k_sel = w.keep(nb)
    assert k_sel == {0.9: 205, 0.5: 1024}[sparsity]
    q = synth.normal_bf16((w.batch, w.num_q_heads, w.head_dim), SEED, w.name + "q", DEV)
    k, v = _kv(w, w.name)
    scores = synth.normal_f32((w.batch, w.num_kv_heads, nb), SEED, w.name + "scores", DEV)
    idx, cnt = _select_on_scores(ctx, w, lens, scores, k_sel)
    want_idx, want_cnt = oracle.select(scores.cpu().numpy(), lens, w.block_size, k_sel * w.block_size, k_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)
    # dense (every output, 10 GFLOP of fp64 on the host) once, at the sparsity the benchmark times
    _decode_and_check(ctx, w, q, k, v, lens, idx, cnt, f"sweep s={sparsity}", dense=(sparsity == 0.9))
