"""Parity at the edges of the supported sizes, through the C ABI: the largest unit count a call
accepts, a one-million-token sequence (more compressed keys than the gate's one-cluster path
holds), and a step on top of it.  Every output is checked against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_08889_b200 import binding, synth
from util import bits, check_attention, ref_sparse, ref_dense

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
THETA = 1.0e6


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def test_largest_unit_count_ragged_short_sequences(ctx):
    # batch * num_kv_heads = 65528 of at most 65535; every unit has one to three blocks
    B, Hq, Hkv, d, b, S = 8191, 16, 8, 128, 64, 192
    # the default workspace is too small for this many units: refused with the size that is needed,
    # which is what seer_workspace_bytes reports up front
    small_shape = binding.make_shape(B, Hq, Hkv, d, b, 0.09)
    need = int(binding.lib().seer_workspace_bytes(small_shape, 0, 0))
    assert need > (64 << 20)
    big = binding.Context(0, workspace_bytes=need)
    try:
        _largest_unit_count(ctx, big, B, Hq, Hkv, d, b, S)
    finally:
        big.close()


def _largest_unit_count(small_ctx, ctx, B, Hq, Hkv, d, b, S):
    lens = synth.np_rng(41, "lens").integers(1, S + 1, size=B).astype(np.int32)
    lens[:4] = [1, 64, 65, 192]
    q = synth.normal_bf16((B, Hq, d), 41, "q", DEV)
    k = synth.normal_bf16((B, Hkv, S, d), 41, "k", DEV)
    v = synth.normal_bf16((B, Hkv, S, d), 41, "v", DEV)
    n = (lens + b - 1) // b
    keep = np.maximum(1, n - 1)
    idx, cnt = synth.random_block_lists(lens, Hkv, b, keep, 3, 41, shuffle=True)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.09)
    lens_t = torch.as_tensor(lens, device=DEV)
    kv = binding.make_kv(k, v, lens_t)
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
    idx_t, cnt_t = torch.as_tensor(idx, device=DEV), torch.as_tensor(cnt, device=DEV)
    with pytest.raises(binding.SeerError) as err:
        small_ctx.seer_sparse_decode(shape, kv, q, idx_t, cnt_t, 3, out, lse)
    assert err.value.status == binding.SEER_ERR_WORKSPACE
    ctx.seer_sparse_decode(shape, kv, q, idx_t, cnt_t, 3, out, lse)
    torch.cuda.synchronize()
    ref = ref_sparse(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.09)
    check_attention(out, lse, *ref, what="65528 units sparse")
    ctx.seer_dense_decode(shape, kv, q, out, lse)
    torch.cuda.synchronize()
    refd = ref_dense(bits(q), bits(k), bits(v), lens, 0.09)
    check_attention(out, lse, *refd, what="65528 units dense")
    assert ctx.device_status() == binding.SEER_OK
    # one more sequence takes the call over the limit: refused on the host, nothing launched
    shape_over = binding.make_shape(B + 1, Hq, Hkv, d, b, 0.09)
    before = ctx.launch_count()
    with pytest.raises(binding.SeerError):
        ctx.seer_dense_decode(shape_over, kv, q, out, lse)
    assert ctx.launch_count() == before


def test_one_million_tokens_gate_select_decode(ctx):
    # 16384 blocks per unit: the gate runs as projection + score/selection kernels, the selection
    # reads its candidates from memory instead of registers, one unit is cut over every CTA
    B, Hq, Hkv, d, dg, b = 1, 8, 2, 128, 128, 64
    L = 1 << 20
    nb = L // b
    q = synth.normal_bf16((B, Hq, d), 42, "q", DEV)
    qn = synth.normal_bf16((B, Hq, d), 42, "qn", DEV)
    k = synth.normal_bf16((B, Hkv, L, d), 42, "k", DEV)
    v = synth.normal_bf16((B, Hkv, L, d), 42, "v", DEV)
    wq = synth.normal_bf16((Hkv, dg, (Hq // Hkv) * d), 42, "wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nb, dg), 42, "kc", DEV)
    lens = np.array([L - 7], np.int32)
    lens_t = torch.as_tensor(lens, device=DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.0884)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nb)
    kv = binding.make_kv(k, v, lens_t)
    max_sel = 1639                                            # s = 0.9 of 16384 blocks
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nb), dtype=torch.float32, device=DEV)
    ctx.seer_gate_select(shape, gate, lens_t, qn, None, max_sel * b, idx, cnt, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    want_sc, _ = oracle.scores(bits(qn), bits(wq), bits(kc), [nb - 1], [int(lens[0]) - 1], THETA)
    got_sc = sc.cpu().numpy()
    assert np.abs(got_sc[0, :, :nb - 1] - want_sc[0, :, :nb - 1]).max() <= 1e-3
    want_idx, want_cnt = oracle.select(got_sc, lens, b, max_sel * b, max_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)
    assert int(cnt[0, 0]) == max_sel and int(idx[0, 0, -1]) == nb - 1
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
    kh, vh = bits(k), bits(v)
    ctx.seer_sparse_decode(shape, kv, q, idx, cnt, max_sel, out, lse)
    torch.cuda.synchronize()
    ref = oracle.sparse(bits(q), kh, vh, lens, want_idx, want_cnt, b, 0.0884)
    check_attention(out, lse, *ref, what="1M tokens sparse", strict=True)
    ctx.seer_dense_decode(shape, kv, q, out, lse)
    torch.cuda.synchronize()
    refd = oracle.dense(bits(q), kh, vh, lens, 0.0884)
    check_attention(out, lse, *refd, what="1M tokens dense", strict=True)
    assert ctx.device_status() == binding.SEER_OK
