"""Parity for sparsity blocks of 16 and 32 tokens (the lower end of the paper's block-size study,
Sec. 5.1): the decode kernel gathers four or two listed blocks into one 64-token tile.  Sparse
decode (contiguous, paged, several query tokens), the compressed-K build and the gate."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_08889_b200 import binding, synth
from util import bits, check_attention, make_qkv, to_paged, ref_sparse, ref_dense, ref_sparse_multi, bf16_ulp

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
THETA = 1.0e6


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def _sparse(ctx, q, k, v, lens, idx, cnt, b, scale, **kw):
    B, Hq, d = q.shape
    shape = binding.make_shape(B, Hq, k.shape[1], d, b, scale)
    lens_t = torch.as_tensor(np.asarray(lens, np.int32), device=DEV)
    kv = binding.make_kv(k, v, lens_t, **kw)
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
    cnt_t = None if cnt is None else torch.as_tensor(cnt, device=DEV)
    ctx.seer_sparse_decode(shape, kv, q, torch.as_tensor(idx, device=DEV).contiguous(), cnt_t, idx.shape[2], out, lse)
    torch.cuda.synchronize()
    return out, lse


@pytest.mark.parametrize("b", [16, 32])
@pytest.mark.parametrize("g,Hkv", [(5, 2), (8, 1), (1, 3)])
def test_sparse_small_blocks_ragged_shuffled_lists(ctx, b, g, Hkv):
    B, d, S = 4, 128, 2048
    Hq = g * Hkv
    # partial last blocks of every flavour: 517 % 16 = 5, 1000 % 32 = 8, one full, one shorter than a block
    lens = np.array([2048, 1000, 517, 7], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 300 + b + g, DEV)
    n = [-(-int(L) // b) for L in lens]
    keep = [max(1, x // 3) for x in n]                  # counts that are not multiples of the blocks per tile
    max_sel = max(keep) + 3
    idx, cnt = synth.random_block_lists(lens, Hkv, b, keep, max_sel, 300 + b, shuffle=True)
    ref = ref_sparse(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.09)
    out, lse = _sparse(ctx, q, k, v, lens, idx, cnt, b, 0.09)
    check_attention(out, lse, *ref, what=f"b={b} g={g}")
    out2, lse2 = _sparse(ctx, q, k, v, lens, idx, None, b, 0.09)          # -1 padding instead of counts
    check_attention(out2, lse2, *ref, what=f"b={b} g={g} no-cnt")
    assert ctx.device_status() == binding.SEER_OK


@pytest.mark.parametrize("b,page_size", [(16, 64), (32, 128)])
def test_sparse_small_blocks_paged_and_split_over_ctas(ctx, b, page_size):
    B, Hq, Hkv, d, S = 2, 8, 2, 128, 16384
    lens = np.array([16384, 12345], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 320 + b, DEV)
    n = [-(-int(L) // b) for L in lens]
    keep = [x // 2 for x in n]
    idx, cnt = synth.random_block_lists(lens, Hkv, b, keep, max(keep), 320 + b)
    ref = oracle.sparse(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.0884)
    out, lse = _sparse(ctx, q, k, v, lens, idx, cnt, b, 0.0884)
    check_attention(out, lse, *ref, what=f"b={b} long", strict=True)
    kp, vp, table = to_paged(k, v, page_size, 320 + b)
    outp, lsep = _sparse(ctx, q, kp, vp, lens, idx, cnt, b, 0.0884, page_table=table, page_size=page_size, max_seq_len=S)
    check_attention(outp, lsep, *ref, what=f"b={b} paged", strict=True)
    assert ctx.device_status() == binding.SEER_OK


@pytest.mark.parametrize("b", [16, 32])
def test_small_blocks_full_selection_is_dense_and_bad_entries_are_flagged(ctx, b):
    B, Hq, Hkv, d, S = 2, 8, 2, 128, 640
    lens = np.array([640, 333], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 340 + b, DEV)
    n = [-(-int(L) // b) for L in lens]
    idx = np.full((B, Hkv, max(n) + 2), -1, np.int32)
    for i in range(B):
        idx[i, :, :n[i]] = np.arange(n[i])
    refd = ref_dense(bits(q), bits(k), bits(v), lens, 0.09)
    out, lse = _sparse(ctx, q, k, v, lens, idx, None, b, 0.09)
    check_attention(out, lse, *refd, what=f"b={b} all blocks")
    assert ctx.device_status() == binding.SEER_OK
    idx[1, 0, 3] = n[1] + 5                                    # past the end: skipped and flagged
    ref = ref_sparse(bits(q), bits(k), bits(v), lens, idx, None, b, 0.09)
    out, lse = _sparse(ctx, q, k, v, lens, idx, None, b, 0.09)
    check_attention(out, lse, *ref, what=f"b={b} bad entry")
    assert ctx.device_status() == binding.SEER_ERR_BAD_INDEX
    assert ctx.device_status() == binding.SEER_OK              # reading the flag clears it


@pytest.mark.parametrize("b,T", [(16, 3), (32, 8), (16, 5)])
def test_small_blocks_several_query_tokens(ctx, b, T):
    B, Hq, Hkv, d, S = 4, 10, 2, 128, 1536
    lens = np.array([1536, 1025, 517, 70], np.int32)          # query tokens straddle block boundaries
    q = synth.normal_bf16((B, T, Hq, d), 360 + b + T, "q", DEV)
    k = synth.normal_bf16((B, Hkv, S, d), 360 + b + T, "k", DEV)
    v = synth.normal_bf16((B, Hkv, S, d), 360 + b + T, "v", DEV)
    n = [-(-int(L) // b) for L in lens]
    keep = [max(2, x // 2) for x in n]
    idx, cnt = synth.random_block_lists(lens, Hkv, b, keep, max(keep) + 1, 360 + b, shuffle=True)
    ref = ref_sparse_multi(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.09)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.09)
    lens_t = torch.as_tensor(lens, device=DEV)
    kv = binding.make_kv(k, v, lens_t)
    out = torch.full((B, T, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, T, Hq), float("nan"), dtype=torch.float32, device=DEV)
    ctx.seer_sparse_decode_multi(shape, kv, q, T, torch.as_tensor(idx, device=DEV), torch.as_tensor(cnt, device=DEV),
                                 idx.shape[2], out, lse)
    torch.cuda.synchronize()
    check_attention(out, lse, *ref, what=f"b={b} T={T}")
    assert ctx.device_status() == binding.SEER_OK


@pytest.mark.parametrize("b", [16, 32])
def test_small_blocks_kcomp_gate_and_step(ctx, b):
    B, Hq, Hkv, d, dg, L = 2, 8, 2, 128, 128, 8192
    nb = L // b
    lens = np.array([L, L - 3 * b], np.int32)                  # both at a block end: the step appends
    q, k, v = make_qkv(B, Hq, Hkv, L, d, 380 + b, DEV)
    qn = synth.normal_bf16((B, Hq, d), 380 + b, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, 4 * d), 380 + b, "wq", DEV, std=0.02)
    wk = synth.normal_bf16((Hkv, dg, 3 * d), 380 + b, "wk", DEV, std=0.02)
    kc = torch.zeros((B, Hkv, nb, dg), dtype=torch.bfloat16, device=DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.0884)
    gate = binding.make_gate(dg, THETA, wq, wk, kc, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    # bulk build of everything but the block that has just filled; the step call appends that one
    ctx.seer_kcomp_append(shape, gate, torch.as_tensor(lens - 1, device=DEV), k, first_block=0, num_blocks=nb)
    kv = binding.make_kv(k, v, lens_t)
    max_sel = nb // 10
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
    ctx.seer_decode_step(shape, kv, gate, q, qn, k, max_sel * b, idx, cnt, max_sel, out, lse)
    torch.cuda.synchronize()
    _, kc_want = oracle.kcomp(bits(k), bits(wk), b, 0, nb, nb, THETA)
    got = synth.bits_to_bf16(bits(kc)).to(torch.float64).numpy()
    for i in range(B):
        n_i = int(lens[i]) // b
        tol = bf16_ulp(kc_want[i, :, :n_i]) + 1e-5 * np.abs(kc_want).max()
        assert (np.abs(got[i, :, :n_i] - kc_want[i, :, :n_i]) <= tol).all()
        assert (got[i, :, n_i:] == 0).all()
    sc = torch.zeros((B, Hkv, nb), dtype=torch.float32, device=DEV)
    idx2, cnt2 = torch.zeros_like(idx), torch.zeros_like(cnt)
    ctx.seer_gate_select(shape, gate, lens_t, qn, None, max_sel * b, idx2, cnt2, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    assert torch.equal(idx, idx2) and torch.equal(cnt, cnt2)
    n = [int(L_) // b for L_ in lens]
    want_sc, _ = oracle.scores(bits(qn), bits(wq), bits(kc), [x - 1 for x in n], [int(L_) - 1 for L_ in lens], THETA)
    got_sc = sc.cpu().numpy()
    for i in range(B):
        assert np.abs(got_sc[i, :, :n[i] - 1] - want_sc[i, :, :n[i] - 1]).max() <= 1e-3
    want_idx, want_cnt = oracle.select(got_sc, lens, b, max_sel * b, max_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)
    ref = oracle.sparse(bits(q), bits(k), bits(v), lens, want_idx, want_cnt, b, 0.0884)
    check_attention(out, lse, *ref, what=f"b={b} step", strict=True)
    assert ctx.device_status() == binding.SEER_OK
