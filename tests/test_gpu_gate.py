"""GPU parity of seer_kcomp_append and seer_gate_select against the fp64 oracle (C ABI).

Stage isolation: each stage's oracle is fed the GPU's output of the stage before it, so a
rounding difference in one stage cannot cascade into a different (equally valid) decision
in the next.  The selection itself is compared bit for bit on identical fp32 scores."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_08889_b200 import binding, synth
from util import bits, check_attention, make_qkv, ref_sparse, kc_tolerance, to_paged

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
THETA = 1.0e6


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def _bf16_ulp_close(got_bits, want_f64):
    got = synth.bits_to_bf16(got_bits).to(torch.float64).numpy()
    bad = np.abs(got - want_f64) > kc_tolerance(want_f64)
    assert not bad.any(), f"{bad.sum()} entries off by more than one ulp; worst {np.abs(got - want_f64).max()}"


@pytest.mark.parametrize("b,dg,token_major", [(64, 128, False), (128, 128, True), (64, 64, False)])
def test_kcomp_bulk_build(ctx, b, dg, token_major):
    B, Hkv, d = 2, 3, 128
    nb = 11
    S = nb * b
    lens = np.array([S, S - b - 5], np.int32)             # second sequence: 9 complete blocks
    if token_major:
        kn = synth.normal_bf16((B, S, Hkv, d), 5, "kn", DEV).permute(0, 2, 1, 3)
    else:
        kn = synth.normal_bf16((B, Hkv, S, d), 5, "kn", DEV)
    wk = synth.normal_bf16((Hkv, dg, 3 * d), 5, "wk", DEV, std=0.02)
    kc = torch.zeros((B, Hkv, nb, dg), dtype=torch.bfloat16, device=DEV)
    shape = binding.make_shape(B, Hkv * 4, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, None, wk, kc, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    ctx.seer_kcomp_append(shape, gate, lens_t, kn, first_block=0, num_blocks=nb)
    torch.cuda.synchronize()
    _, want = oracle.kcomp(bits(kn), bits(wk), b, 0, nb, nb, THETA)
    got = bits(kc)
    _bf16_ulp_close(got[0], want[0])
    _bf16_ulp_close(got[1, :, :9], want[1, :, :9])
    assert np.all(got[1, :, 9:] == 0)                     # incomplete blocks are not written
    # a sub-range only touches its own entries
    kc2 = torch.zeros_like(kc)
    gate2 = binding.make_gate(dg, THETA, None, wk, kc2, nb)
    ctx.seer_kcomp_append(shape, gate2, lens_t, kn, first_block=3, num_blocks=5)
    torch.cuda.synchronize()
    got2 = bits(kc2)
    assert np.array_equal(got2[:, :, 3:8], got[:, :, 3:8])
    assert np.all(got2[:, :, :3] == 0) and np.all(got2[:, :, 8:] == 0)


@pytest.mark.parametrize("dg,token_major,first", [(128, False, 0), (64, True, 0), (128, True, 37)])
def test_kcomp_bulk_build_large_enough_for_the_streaming_kernel(ctx, dg, token_major, first):
    """From 2 * (SM count) work items of 16 blocks on (block size 64, d_gate <= 128) the bulk build runs as
    the persistent kernel with a ring of stages and specialised warps: 3 x 4 units x 26 groups = 312 items
    here, ragged lengths (one sequence ends inside a group, one has a single group), four heads (a CTA
    changes W_k slice several times), both K layouts, and a build that starts in the middle of a group."""
    B, Hkv, d, b = 3, 4, 128, 64
    nb = 416
    S = nb * b
    lens = np.array([S, 333 * b + 17, 9 * b], np.int32)
    n_complete = [nb, 333, 9]
    if token_major:
        kn = synth.normal_bf16((B, S, Hkv, d), 6, "kn", DEV).permute(0, 2, 1, 3)
    else:
        kn = synth.normal_bf16((B, Hkv, S, d), 6, "kn", DEV)
    wk = synth.normal_bf16((Hkv, dg, 3 * d), 6, "wk", DEV, std=0.02)
    kc = torch.zeros((B, Hkv, nb, dg), dtype=torch.bfloat16, device=DEV)
    shape = binding.make_shape(B, Hkv * 2, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, None, wk, kc, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    for _ in range(2):                                    # the second launch overlaps the first one's tail
        ctx.seer_kcomp_append(shape, gate, lens_t, kn, first_block=first, num_blocks=nb - first)
    torch.cuda.synchronize()
    assert ctx.device_status() == binding.SEER_OK
    _, want = oracle.kcomp(bits(kn), bits(wk), b, 0, nb, nb, THETA)
    got = bits(kc)
    for i in range(B):
        if n_complete[i] > first:
            _bf16_ulp_close(got[i, :, first:n_complete[i]], want[i, :, first:n_complete[i]])
        assert np.all(got[i, :, max(first, n_complete[i]):] == 0)     # incomplete blocks are not written
        assert np.all(got[i, :, :first] == 0)             # nor blocks before the first one asked for


def test_kcomp_bulk_build_more_sequences_than_the_length_cache_holds(ctx):
    """The streaming bulk build keeps the first 2048 sequence lengths in shared memory and reads the others from
    global memory: 2100 sequences of one KV head, 16 blocks each (2100 work items), lengths that differ on both
    sides of that boundary."""
    B, Hkv, d, b, dg = 2100, 1, 128, 64, 128
    nb = 16
    S = nb * b
    lens = np.full(B, S, np.int32)
    lens[5] = 3 * b + 1
    lens[2047] = 7 * b
    lens[2048] = 2 * b + 63
    lens[2099] = 11 * b
    kn = synth.normal_bf16((B, Hkv, S, d), 8, "kn", DEV)
    wk = synth.normal_bf16((Hkv, dg, 3 * d), 8, "wk", DEV, std=0.02)
    kc = torch.zeros((B, Hkv, nb, dg), dtype=torch.bfloat16, device=DEV)
    shape = binding.make_shape(B, Hkv * 4, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, None, wk, kc, nb)
    ctx.seer_kcomp_append(shape, gate, torch.as_tensor(lens, device=DEV), kn, first_block=0, num_blocks=nb)
    torch.cuda.synchronize()
    assert ctx.device_status() == binding.SEER_OK
    got = bits(kc)
    for i in (0, 5, 2046, 2047, 2048, 2049, 2099):
        _, want = oracle.kcomp(bits(kn[i:i + 1]), bits(wk), b, 0, nb, nb, THETA)
        n = int(lens[i]) // b
        _bf16_ulp_close(got[i, :, :n], want[0, :, :n])
        assert np.all(got[i, :, n:] == 0)


def test_kcomp_append_when_a_block_fills(ctx):
    B, Hkv, d, dg, b, nb = 3, 2, 128, 128, 64, 8
    lens = np.array([5 * b, 5 * b + 1, 3 * b], np.int32)  # sequences 0 and 2 just filled a block
    kn = synth.normal_bf16((B, Hkv, nb * b, d), 6, "kn", DEV)
    wk = synth.normal_bf16((Hkv, dg, 3 * d), 6, "wk", DEV, std=0.02)
    kc = torch.zeros((B, Hkv, nb, dg), dtype=torch.bfloat16, device=DEV)
    shape = binding.make_shape(B, Hkv * 4, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, None, wk, kc, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    ctx.seer_kcomp_append(shape, gate, lens_t, kn)        # first_block = -1
    torch.cuda.synchronize()
    _, want = oracle.kcomp(bits(kn), bits(wk), b, 0, nb, nb, THETA)
    got = bits(kc)
    _bf16_ulp_close(got[0, :, 4], want[0, :, 4])
    _bf16_ulp_close(got[2, :, 2], want[2, :, 2])
    mask = np.ones((B, nb), bool); mask[0, 4] = False; mask[2, 2] = False
    assert np.all(got.transpose(0, 2, 1, 3)[mask] == 0)
    # the same update from a rolling window that holds only the block being appended
    win = torch.stack([kn[0, :, 4 * b:5 * b], kn[1, :, 4 * b:5 * b], kn[2, :, 2 * b:3 * b]]).contiguous()
    kc3 = torch.zeros_like(kc)
    gate3 = binding.make_gate(dg, THETA, None, wk, kc3, nb)
    ctx.seer_kcomp_append(shape, gate3, lens_t, win, rows_block_local=True)
    torch.cuda.synchronize()
    assert np.array_equal(bits(kc3), got)


@pytest.mark.parametrize("g,b", [(4, 64), (5, 64), (8, 128), (1, 64)])
def test_gate_scores_and_selection(ctx, g, b):
    B, Hkv, d, dg = 3, 2, 128, 128
    Hq = g * Hkv
    nbmax = 40
    lens = np.array([nbmax * b, 17 * b + 9, 2 * b - 1], np.int32)
    qn = synth.normal_bf16((B, Hq, d), 8, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, g * d), 8, "wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nbmax, dg), 8, "kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nbmax)
    lens_t = torch.as_tensor(lens, device=DEV)
    max_sel = 12
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nbmax), dtype=torch.float32, device=DEV)
    budget = 7 * b
    ctx.seer_gate_select(shape, gate, lens_t, qn, None, budget, idx, cnt, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    n = [-(-int(L) // b) for L in lens]
    want_sc, _ = oracle.scores(bits(qn), bits(wq), bits(kc), [x - 1 for x in n], [int(L) - 1 for L in lens], THETA)
    got_sc = sc.cpu().numpy()
    for i in range(B):
        assert np.abs(got_sc[i, :, :n[i] - 1] - want_sc[i, :, :n[i] - 1]).max() <= 1e-3
    # selection is exact on the scores the GPU itself produced
    want_idx, want_cnt = oracle.select(got_sc, lens, b, budget, max_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx)
    assert np.array_equal(cnt.cpu().numpy(), want_cnt)
    # without scores_out the internal scratch gives the same lists
    idx2 = torch.zeros_like(idx); cnt2 = torch.zeros_like(cnt)
    ctx.seer_gate_select(shape, gate, lens_t, qn, None, budget, idx2, cnt2, max_sel)
    torch.cuda.synchronize()
    assert torch.equal(idx, idx2) and torch.equal(cnt, cnt2)


@pytest.mark.parametrize("nbmax,dg,g", [(6000, 128, 2), (8192, 256, 1), (5000, 64, 4)])
def test_gate_largest_clusters_several_key_batches_per_cta(ctx, nbmax, dg, g):
    # 4097..8192 compressed keys per unit: clusters of 8 CTAs, three or more key batches per CTA
    # (staged, registers, staged again ...), candidates of the selection read from shared memory
    B, Hkv, d, b = 2, 2, 128, 64
    Hq = g * Hkv
    lens = np.array([nbmax * b, (nbmax - 700) * b + 5], np.int32)
    qn = synth.normal_bf16((B, Hq, d), 19, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, g * d), 19, "wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nbmax, dg), 19, "kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nbmax)
    lens_t = torch.as_tensor(lens, device=DEV)
    max_sel = 600
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nbmax), dtype=torch.float32, device=DEV)
    before = ctx.launch_count()
    ctx.seer_gate_select(shape, gate, lens_t, qn, None, max_sel * b, idx, cnt, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    assert ctx.launch_count() - before == 1
    n = [-(-int(L) // b) for L in lens]
    want_sc, _ = oracle.scores(bits(qn), bits(wq), bits(kc), [x - 1 for x in n], [int(L) - 1 for L in lens], THETA)
    got_sc = sc.cpu().numpy()
    for i in range(B):
        assert np.abs(got_sc[i, :, :n[i] - 1] - want_sc[i, :, :n[i] - 1]).max() <= 1e-3
    want_idx, want_cnt = oracle.select(got_sc, lens, b, max_sel * b, max_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)
    # several query tokens on the same size
    T = 3
    qn3 = synth.normal_bf16((B, T, Hq, d), 19, "qn3", DEV)
    ctx.seer_gate_select_multi(shape, gate, lens_t, qn3, None, T, max_sel * b, idx, cnt, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    got_sc = sc.cpu().numpy()
    want_sc = oracle.scores_multi(bits(qn3), bits(wq), bits(kc), lens, b, THETA)
    for i in range(B):
        jf = (int(lens[i]) - T) // b
        assert np.abs(got_sc[i, :, :jf] - want_sc[i, :, :jf]).max() <= 1e-3
    want_idx, want_cnt = oracle.select_multi(got_sc, lens, b, max_sel * b, T, max_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)
    assert ctx.device_status() == binding.SEER_OK


def test_gate_more_keys_than_one_cluster_holds(ctx):
    # above 8192 compressed keys per unit the gate runs as projection + score/selection kernels
    B, Hkv, g, d, dg, b = 1, 2, 2, 128, 64, 64
    Hq = g * Hkv
    nbmax = 9000
    lens = np.array([nbmax * b - 5], np.int32)
    qn = synth.normal_bf16((B, Hq, d), 18, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, g * d), 18, "wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nbmax, dg), 18, "kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nbmax)
    lens_t = torch.as_tensor(lens, device=DEV)
    max_sel = 900
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nbmax), dtype=torch.float32, device=DEV)
    before = ctx.launch_count()
    ctx.seer_gate_select(shape, gate, lens_t, qn, None, max_sel * b, idx, cnt, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    assert ctx.launch_count() - before == 2
    want_sc, _ = oracle.scores(bits(qn), bits(wq), bits(kc), [nbmax - 1], [int(lens[0]) - 1], THETA)
    got_sc = sc.cpu().numpy()
    assert np.abs(got_sc[0, :, :nbmax - 1] - want_sc[0, :, :nbmax - 1]).max() <= 1e-3
    want_idx, want_cnt = oracle.select(got_sc, lens, b, max_sel * b, max_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)


@pytest.mark.parametrize("case", ["normal", "ties", "all_equal", "specials"])
@pytest.mark.parametrize("b", [64, 128])
def test_selection_bit_exact_on_given_scores(ctx, case, b):
    B, Hkv, nbmax = 4, 3, 700
    r = synth.np_rng(9, case)
    sc = r.normal(size=(B, Hkv, nbmax)).astype(np.float32)
    if case == "ties":
        sc = np.round(sc * 4) / 4
    elif case == "all_equal":
        sc[:] = 0.5
    elif case == "specials":
        sc[:, :, ::7] = 0.0
        sc[:, :, 3::11] = -0.0
        sc[:, :, 5::13] = np.nan
        sc[:, :, 6::17] = -np.inf
        sc[:, :, 8::19] = np.inf
    lens = np.array([nbmax * b, 333 * b + 1, b, 2 * b], np.int32)
    shape = binding.make_shape(B, Hkv * 4, Hkv, 128, b, 0.1)
    gate = binding.make_gate(128, THETA, None, None, None, nbmax)
    lens_t = torch.as_tensor(lens, device=DEV)
    sc_t = torch.as_tensor(sc, device=DEV)
    for budget, max_sel in [(64 * b, 64), (b, 8), (0, 8), (700 * b, 700), (650 * b, 700), (300 * b, 100)]:
        idx = torch.full((B, Hkv, max_sel), 77, dtype=torch.int32, device=DEV)
        cnt = torch.full((B, Hkv), 77, dtype=torch.int32, device=DEV)
        ctx.seer_gate_select(shape, gate, lens_t, None, sc_t, budget, idx, cnt, max_sel)
        torch.cuda.synchronize()
        want_idx, want_cnt = oracle.select(sc, lens, b, budget, max_sel)
        assert np.array_equal(cnt.cpu().numpy(), want_cnt), (case, budget)
        assert np.array_equal(idx.cpu().numpy(), want_idx), (case, budget)


def test_gate_then_decode_end_to_end_14b_shape_small(ctx):
    # K_nope := K cache, bulk build of the compressed keys, gate, selection, sparse decode
    B, Hq, Hkv, d, dg, b = 2, 10, 2, 128, 128, 64
    nb = 48
    S = nb * b
    lens = np.array([S, S - 3 * b - 7], np.int32)
    q = synth.normal_bf16((B, Hq, d), 12, "q", DEV)
    qn = synth.normal_bf16((B, Hq, d), 12, "qn", DEV)
    k = synth.normal_bf16((B, Hkv, S, d), 12, "k", DEV)
    v = synth.normal_bf16((B, Hkv, S, d), 12, "v", DEV)
    wq = synth.normal_bf16((Hkv, dg, 5 * d), 12, "wq", DEV, std=0.02)
    wk = synth.normal_bf16((Hkv, dg, 3 * d), 12, "wk", DEV, std=0.02)
    kc = torch.zeros((B, Hkv, nb, dg), dtype=torch.bfloat16, device=DEV)
    scale = 1.0 / np.sqrt(d)
    shape = binding.make_shape(B, Hq, Hkv, d, b, scale)
    gate = binding.make_gate(dg, THETA, wq, wk, kc, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    max_sel = 8
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nb), dtype=torch.float32, device=DEV)
    out = torch.zeros((B, Hq, d), dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros((B, Hq), dtype=torch.float32, device=DEV)
    kv = binding.make_kv(k, v, lens_t)
    ctx.seer_kcomp_append(shape, gate, lens_t, k, first_block=0, num_blocks=nb)
    ctx.seer_gate_select(shape, gate, lens_t, qn, None, max_sel * b, idx, cnt, max_sel, scores_out=sc)
    ctx.seer_sparse_decode(shape, kv, q, idx, cnt, max_sel, out, lse)
    torch.cuda.synchronize()
    # stage 1: compressed keys
    _, kc_want = oracle.kcomp(bits(k), bits(wk), b, 0, nb, nb, THETA)
    got_kc = bits(kc)
    _bf16_ulp_close(got_kc[0], kc_want[0])
    _bf16_ulp_close(got_kc[1, :, :44], kc_want[1, :, :44])
    # stage 2: scores on the GPU's compressed keys
    n = [-(-int(L) // b) for L in lens]
    want_sc, _ = oracle.scores(bits(qn), bits(wq), got_kc, [x - 1 for x in n], [int(L) - 1 for L in lens], THETA)
    got_sc = sc.cpu().numpy()
    for i in range(B):
        assert np.abs(got_sc[i, :, :n[i] - 1] - want_sc[i, :, :n[i] - 1]).max() <= 1e-3
    # stage 3: selection on the GPU's scores, exact
    want_idx, want_cnt = oracle.select(got_sc, lens, b, max_sel * b, max_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)
    # stage 4: attention over the GPU's lists
    ref = ref_sparse(bits(q), bits(k), bits(v), lens, want_idx, want_cnt, b, scale)
    check_attention(out, lse, *ref, what="end to end")
    assert ctx.device_status() == binding.SEER_OK


def test_single_call_step_equals_the_three_calls(ctx):
    B, Hq, Hkv, d, dg, b = 3, 8, 2, 128, 128, 64
    nb = 40
    S = nb * b
    lens = np.array([S, S - b, 17 * b + 3], np.int32)          # sequences 0 and 1 have just filled a block
    q = synth.normal_bf16((B, Hq, d), 21, "q", DEV)
    qn = synth.normal_bf16((B, Hq, d), 21, "qn", DEV)
    k = synth.normal_bf16((B, Hkv, S, d), 21, "k", DEV)
    v = synth.normal_bf16((B, Hkv, S, d), 21, "v", DEV)
    wq = synth.normal_bf16((Hkv, dg, 4 * d), 21, "wq", DEV, std=0.02)
    wk = synth.normal_bf16((Hkv, dg, 3 * d), 21, "wk", DEV, std=0.02)
    scale = 1.0 / np.sqrt(d)
    shape = binding.make_shape(B, Hq, Hkv, d, b, scale)
    lens_t = torch.as_tensor(lens, device=DEV)
    kv = binding.make_kv(k, v, lens_t)
    max_sel = 6
    res = []
    for fused in (False, True):
        kc = synth.normal_bf16((B, Hkv, nb, dg), 21, "kc", DEV)     # "earlier" entries
        gate = binding.make_gate(dg, THETA, wq, wk, kc, nb)
        idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
        cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
        out = torch.zeros((B, Hq, d), dtype=torch.bfloat16, device=DEV)
        lse = torch.zeros((B, Hq), dtype=torch.float32, device=DEV)
        if fused:
            ctx.seer_decode_step(shape, kv, gate, q, qn, k, max_sel * b, idx, cnt, max_sel, out, lse)
        else:
            ctx.seer_kcomp_append(shape, gate, lens_t, k)
            ctx.seer_gate_select(shape, gate, lens_t, qn, None, max_sel * b, idx, cnt, max_sel)
            ctx.seer_sparse_decode(shape, kv, q, idx, cnt, max_sel, out, lse)
        torch.cuda.synchronize()
        res.append((kc, idx, cnt, out, lse))
    for a, c in zip(res[0], res[1]):
        assert torch.equal(a, c)
    assert ctx.device_status() == binding.SEER_OK


@pytest.mark.parametrize("tau", [0.002, 0.006, 0.05])
def test_threshold_selection(ctx, tau):
    # the decision is a floating-point comparison (fp32 on the GPU, fp64 in the oracle): blocks
    # whose probability is not within rounding of tau must agree exactly, the few others may differ
    B, Hkv, b, nbmax, max_sel = 4, 3, 64, 700, 700
    r = synth.np_rng(31, "thr")
    sc = (r.normal(size=(B, Hkv, nbmax)) * 1.5).astype(np.float32)
    lens = np.array([nbmax * b, 333 * b + 1, b, 2 * b], np.int32)
    shape = binding.make_shape(B, Hkv * 4, Hkv, 128, b, 0.1)
    gate = binding.make_gate(128, THETA, None, None, None, nbmax)
    lens_t = torch.as_tensor(lens, device=DEV)
    idx = torch.full((B, Hkv, max_sel), 77, dtype=torch.int32, device=DEV)
    cnt = torch.full((B, Hkv), 77, dtype=torch.int32, device=DEV)
    ctx.seer_gate_select_threshold(shape, gate, lens_t, None, torch.as_tensor(sc, device=DEV), tau, idx, cnt, max_sel)
    torch.cuda.synchronize()
    want_idx, want_cnt, probs = oracle.select_threshold(sc, lens, b, tau, max_sel)
    idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
    total = 0
    for i in range(B):
        n = -(-int(lens[i]) // b)
        for h in range(Hkv):
            got = set(idx[i, h, :cnt[i, h]].tolist())
            want = set(want_idx[i, h, :want_cnt[i, h]].tolist())
            assert n - 1 in got and list(idx[i, h, :cnt[i, h]]) == sorted(got)
            assert np.all(idx[i, h, cnt[i, h]:] == -1)
            for j in got ^ want:
                assert abs(probs[i, h, j] - tau) <= 1e-5 * tau + 1e-9, (i, h, j, probs[i, h, j])
            total += len(got)
    assert total > B * Hkv                                   # the threshold did select something
    # too small a list: the highest-scoring max_sel-1 are kept, exactly as the budget method would
    small = 9
    idx2 = torch.zeros((B, Hkv, small), dtype=torch.int32, device=DEV)
    cnt2 = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    ctx.seer_gate_select_threshold(shape, gate, lens_t, None, torch.as_tensor(sc, device=DEV), 1e-7, idx2, cnt2, small)
    torch.cuda.synchronize()
    w2, c2, _ = oracle.select_threshold(sc, lens, b, 1e-7, small)
    assert np.array_equal(idx2.cpu().numpy(), w2) and np.array_equal(cnt2.cpu().numpy(), c2)
    with pytest.raises(binding.SeerError):
        ctx.seer_gate_select_threshold(shape, gate, lens_t, None, torch.as_tensor(sc, device=DEV), 1.5, idx2, cnt2, small)


@pytest.mark.parametrize("nbmax,tau,max_sel", [(700, 2e-3, 700), (9000, 1.5e-4, 4000)])
def test_threshold_selection_on_scores_the_gate_computes(ctx, nbmax, tau, max_sel):
    # the threshold method through both scoring paths: the one-kernel gate (up to 8192 compressed
    # keys per unit) and the projection + score/selection pair above that.  Scores against the
    # oracle; the selection against the oracle's threshold rule applied to the GPU's own scores,
    # where only blocks whose probability is within rounding of tau may fall on either side.
    B, Hkv, g, d, dg, b = 2, 2, 4, 128, 128, 64
    Hq = g * Hkv
    lens = np.array([nbmax * b - 5, (nbmax // 2) * b + 1], np.int32)
    qn = synth.normal_bf16((B, Hq, d), 41, "thr:qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, g * d), 41, "thr:wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nbmax, dg), 41, "thr:kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nbmax)
    lens_t = torch.as_tensor(lens, device=DEV)
    idx = torch.full((B, Hkv, max_sel), 77, dtype=torch.int32, device=DEV)
    cnt = torch.full((B, Hkv), 77, dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nbmax), dtype=torch.float32, device=DEV)
    ctx.seer_gate_select_threshold(shape, gate, lens_t, qn, None, tau, idx, cnt, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    n = [-(-int(L) // b) for L in lens]
    want_sc, _ = oracle.scores(bits(qn), bits(wq), bits(kc), [x - 1 for x in n], [int(L) - 1 for L in lens], THETA)
    got_sc = sc.cpu().numpy()
    for i in range(B):
        assert np.abs(got_sc[i, :, :n[i] - 1] - want_sc[i, :, :n[i] - 1]).max() <= 1e-3
    want_idx, want_cnt, probs = oracle.select_threshold(got_sc, lens, b, tau, max_sel)
    idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
    total = 0
    for i in range(B):
        for h in range(Hkv):
            got = set(idx[i, h, :cnt[i, h]].tolist())
            want = set(want_idx[i, h, :want_cnt[i, h]].tolist())
            assert n[i] - 1 in got and list(idx[i, h, :cnt[i, h]]) == sorted(got)
            assert np.all(idx[i, h, cnt[i, h]:] == -1)
            for j in got ^ want:
                assert abs(probs[i, h, j] - tau) <= 1e-5 * tau + 1e-9, (i, h, j, probs[i, h, j])
            total += len(got)
            assert 1 < len(got) < n[i]                       # the threshold cut somewhere inside
    # without scores_out (scores stay in the library's scratch) the lists are the same
    idx2 = torch.full((B, Hkv, max_sel), 55, dtype=torch.int32, device=DEV)
    cnt2 = torch.full((B, Hkv), 55, dtype=torch.int32, device=DEV)
    ctx.seer_gate_select_threshold(shape, gate, lens_t, qn, None, tau, idx2, cnt2, max_sel)
    torch.cuda.synchronize()
    assert np.array_equal(idx2.cpu().numpy(), idx) and np.array_equal(cnt2.cpu().numpy(), cnt)
    assert ctx.device_status() == binding.SEER_OK


@pytest.mark.parametrize("b", [16, 64, 128])
def test_step_call_on_ragged_lengths_budget_above_and_below_the_block_counts(ctx, b):
    # the step call on sequences shorter than the budget, empty ones, one block only
    B, Hq, Hkv, d, dg, S = 6, 8, 2, 128, 128, 4096
    nb = S // b
    lens = np.array([S, (nb * 5 // 8) * b + 3, 5 * b, b, 7, 0], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 77 + b, DEV)
    qn = synth.normal_bf16((B, Hq, d), 77 + b, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, 4 * d), 77 + b, "wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nb, dg), 77 + b, "kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.0884)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    kv = binding.make_kv(k, v, lens_t)
    for budget, max_sel in [(12 * b, 12), (12 * b, 9), (b, 4), (0, 3), (1000 * b, nb)]:
        idx = torch.full((B, Hkv, max_sel), 55, dtype=torch.int32, device=DEV)
        cnt = torch.full((B, Hkv), 55, dtype=torch.int32, device=DEV)
        out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
        lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
        ctx.seer_decode_step(shape, kv, gate, q, qn, None, budget, idx, cnt, max_sel, out, lse)
        torch.cuda.synchronize()
        sc = torch.zeros((B, Hkv, nb), dtype=torch.float32, device=DEV)
        idx2, cnt2 = torch.zeros_like(idx), torch.zeros_like(cnt)
        ctx.seer_gate_select(shape, gate, lens_t, qn, None, budget, idx2, cnt2, max_sel, scores_out=sc)
        torch.cuda.synchronize()
        assert torch.equal(idx, idx2) and torch.equal(cnt, cnt2)
        want_idx, want_cnt = oracle.select(sc.cpu().numpy(), lens, b, budget, max_sel)
        assert np.array_equal(cnt.cpu().numpy(), want_cnt) and np.array_equal(idx.cpu().numpy(), want_idx)
        ref = ref_sparse(bits(q), bits(k), bits(v), lens, want_idx, want_cnt, b, 0.0884)
        check_attention(out, lse, *ref, what=f"step b={b} budget={budget}")
    assert ctx.device_status() == binding.SEER_OK


def test_step_call_on_a_paged_cache_with_ragged_lengths(ctx):
    """seer_decode_step over a paged K/V pool (pages of 128 tokens under a random permutation) and ragged
    lengths: inside the step the attention kernel counts its tiles from the sequence lengths before the gate
    has finished, so the lists, the counts and the attention are checked against the oracle for budgets above
    and below the sequences' block counts."""
    B, Hq, Hkv, d, dg, S, b = 5, 10, 2, 128, 128, 4096, 64
    nb = S // b
    lens = np.array([S, 37 * b + 9, 3 * b, b + 1, 0], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 91, DEV)
    kp, vp, table = to_paged(k, v, 128, 91)
    qn = synth.normal_bf16((B, Hq, d), 91, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, 5 * d), 91, "wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nb, dg), 91, "kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.0884)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    kv = binding.make_kv(kp, vp, lens_t, max_seq_len=S, page_table=table, page_size=128)
    for budget, max_sel in [(20 * b, 20), (20 * b, 6), (2 * b, 8)]:
        idx = torch.full((B, Hkv, max_sel), 55, dtype=torch.int32, device=DEV)
        cnt = torch.full((B, Hkv), 55, dtype=torch.int32, device=DEV)
        out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
        lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
        for _ in range(2):                                  # (the second call's kernels overlap the first's)
            ctx.seer_decode_step(shape, kv, gate, q, qn, None, budget, idx, cnt, max_sel, out, lse)
        torch.cuda.synchronize()
        sc = torch.zeros((B, Hkv, nb), dtype=torch.float32, device=DEV)
        idx2, cnt2 = torch.zeros_like(idx), torch.zeros_like(cnt)
        ctx.seer_gate_select(shape, gate, lens_t, qn, None, budget, idx2, cnt2, max_sel, scores_out=sc)
        torch.cuda.synchronize()
        want_idx, want_cnt = oracle.select(sc.cpu().numpy(), lens, b, budget, max_sel)
        assert np.array_equal(cnt.cpu().numpy(), want_cnt) and np.array_equal(idx.cpu().numpy(), want_idx)
        ref = ref_sparse(bits(q), bits(k), bits(v), lens, want_idx, want_cnt, b, 0.0884)
        check_attention(out, lse, *ref, what=f"paged step budget={budget}")
    assert ctx.device_status() == binding.SEER_OK


def test_steps_back_to_back_with_and_without_the_list_marks(monkeypatch):
    """Many seer_decode_step calls in a row without a synchronisation, the queries alternating between two
    draws (so that consecutive steps select different blocks and a mark or a list left by an earlier step
    would give a wrong result), on ragged lengths: every step's lists are the oracle's selection on the
    scores the gate computes, every output the oracle's attention over those lists -- with the per-unit
    marks between the gate and the attention kernel (default) and with SEER_STEP_LIST_FLAGS=0."""
    B, Hq, Hkv, d, dg, b, S = 4, 8, 2, 128, 128, 64, 8192
    nb = S // b
    lens = np.array([S, S - 5 * b - 9, 40 * b + 1, 3 * b], np.int32)
    _, k, v = make_qkv(B, Hq, Hkv, S, d, 91, DEV)
    qs = [synth.normal_bf16((B, Hq, d), 91, f"q{j}", DEV) for j in range(2)]
    qns = [synth.normal_bf16((B, Hq, d), 91, f"qn{j}", DEV) for j in range(2)]
    wq = synth.normal_bf16((Hkv, dg, 4 * d), 91, "wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nb, dg), 91, "kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.0884)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    kv = binding.make_kv(k, v, lens_t)
    budget, max_sel, steps = 24 * b, 24, 16

    def run(c):
        # what each of the two query draws must give: scores from the gate alone, the rest from the oracle
        want = []
        for j in range(2):
            sc = torch.zeros((B, Hkv, nb), dtype=torch.float32, device=DEV)
            i0 = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
            c0 = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
            c.seer_gate_select(shape, gate, lens_t, qns[j], None, budget, i0, c0, max_sel, scores_out=sc)
            torch.cuda.synchronize()
            w_idx, w_cnt = oracle.select(sc.cpu().numpy(), lens, b, budget, max_sel)
            want.append((w_idx, w_cnt, ref_sparse(bits(qs[j]), bits(k), bits(v), lens, w_idx, w_cnt, b, 0.0884)))
        assert not np.array_equal(want[0][0], want[1][0])          # the two draws do select differently
        idx = [torch.full((B, Hkv, max_sel), 55, dtype=torch.int32, device=DEV) for _ in range(steps)]
        cnt = [torch.full((B, Hkv), 55, dtype=torch.int32, device=DEV) for _ in range(steps)]
        outs = [torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV) for _ in range(steps)]
        lses = [torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV) for _ in range(steps)]
        shared_idx = torch.full((B, Hkv, max_sel), 55, dtype=torch.int32, device=DEV)
        shared_cnt = torch.full((B, Hkv), 55, dtype=torch.int32, device=DEV)
        torch.cuda.synchronize()
        for s in range(steps):
            # even steps reuse one list buffer (each gate overwrites the lists the previous attention read),
            # odd steps have their own, kept for the comparison
            li, lc = (shared_idx, shared_cnt) if s % 4 == 0 else (idx[s], cnt[s])
            c.seer_decode_step(shape, kv, gate, qs[s & 1], qns[s & 1], None, budget, li, lc, max_sel, outs[s], lses[s])
        torch.cuda.synchronize()
        for s in range(steps):
            w_idx, w_cnt, (o_w, l_w, a_w) = want[s & 1]
            if s % 4 != 0:
                assert np.array_equal(idx[s].cpu().numpy(), w_idx) and np.array_equal(cnt[s].cpu().numpy(), w_cnt), s
            check_attention(outs[s], lses[s], o_w, l_w, a_w, what=f"step {s}")
        assert c.device_status() == binding.SEER_OK

    with_marks = binding.Context(0)
    try:
        run(with_marks)
    finally:
        with_marks.close()
    monkeypatch.setenv("SEER_STEP_LIST_FLAGS", "0")             # read when a context is created
    without = binding.Context(0)
    try:
        run(without)
    finally:
        without.close()
