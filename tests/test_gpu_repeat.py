"""The same call repeated a few thousand times: work stealing and the in-kernel combine make the
order of the floating-point merges vary from launch to launch, never the set of tiles.  Every
repetition must stay within the parity bound of the oracle result; the gate's lists must be
identical every time (the selection is exact)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_08889_b200 import binding, synth
from util import bits, check_attention, make_qkv, ref_sparse_multi

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("T", [1, 3])
def test_sparse_decode_repeated_launches_agree(ctx, T):
    B, Hq, Hkv, d, b, S = 2, 40, 8, 128, 64, 32768
    lens = np.array([S, S - 1234], np.int32)
    q = synth.normal_bf16((B, T, Hq, d), 501, "q", DEV)
    k = synth.normal_bf16((B, Hkv, S, d), 501, "k", DEV)
    v = synth.normal_bf16((B, Hkv, S, d), 501, "v", DEV)
    n = [-(-int(L) // b) for L in lens]
    keep = [x // 2 for x in n]
    idx, cnt = synth.random_block_lists(lens, Hkv, b, keep, max(keep), 501)
    ref_o, ref_l = oracle.sparse_multi(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.0884)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.0884)
    lens_t = torch.as_tensor(lens, device=DEV)
    kv = binding.make_kv(k, v, lens_t)
    idx_t, cnt_t = torch.as_tensor(idx, device=DEV), torch.as_tensor(cnt, device=DEV)
    out = torch.empty((B, T, Hq, d), dtype=torch.bfloat16, device=DEV)
    lse = torch.empty((B, T, Hq), dtype=torch.float32, device=DEV)
    ctx.seer_sparse_decode_multi(shape, kv, q, T, idx_t, cnt_t, idx.shape[2], out, lse)
    torch.cuda.synchronize()
    check_attention(out, lse, ref_o, ref_l, what="first launch", strict=True)
    first_o, first_l = out.float().clone(), lse.clone()
    worst_o = torch.zeros((), device=DEV)
    worst_l = torch.zeros((), device=DEV)
    for rep in range(1500):
        out.fill_(float("nan"))
        lse.fill_(float("nan"))
        ctx.seer_sparse_decode_multi(shape, kv, q, T, idx_t, cnt_t, idx.shape[2], out, lse)
        worst_o = torch.maximum(worst_o, (out.float() - first_o).abs().nan_to_num(nan=1e9).max())
        worst_l = torch.maximum(worst_l, (lse - first_l).abs().nan_to_num(nan=1e9).max())
    torch.cuda.synchronize()
    # bf16 outputs of magnitude < 0.25 differ by a few units in the last place at most
    assert float(worst_o) <= 2e-3 and float(worst_l) <= 1e-4, (float(worst_o), float(worst_l))
    assert ctx.device_status() == binding.SEER_OK


def test_gate_repeated_launches_give_identical_lists(ctx):
    B, Hq, Hkv, d, dg, b, nb = 4, 40, 8, 128, 128, 64, 2048
    lens = np.array([nb * b, nb * b - 77, 1000 * b, 64 * b + 1], np.int32)
    qn = synth.normal_bf16((B, Hq, d), 502, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, 5 * d), 502, "wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nb, dg), 502, "kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, 1.0e6, wq, None, kc, nb)
    lens_t = torch.as_tensor(lens, device=DEV)
    max_sel = 205
    idx = torch.zeros((B, Hkv, max_sel), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nb), dtype=torch.float32, device=DEV)
    ctx.seer_gate_select(shape, gate, lens_t, qn, None, max_sel * b, idx, cnt, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    want_idx, want_cnt = oracle.select(sc.cpu().numpy(), lens, b, max_sel * b, max_sel)
    assert np.array_equal(idx.cpu().numpy(), want_idx) and np.array_equal(cnt.cpu().numpy(), want_cnt)
    first_idx, first_cnt, first_sc = idx.clone(), cnt.clone(), sc.clone()
    bad = torch.zeros((), dtype=torch.int64, device=DEV)
    for rep in range(1500):
        idx.fill_(-7)
        cnt.fill_(-7)
        ctx.seer_gate_select(shape, gate, lens_t, qn, None, max_sel * b, idx, cnt, max_sel, scores_out=sc)
        bad += (idx != first_idx).sum() + (cnt != first_cnt).sum() + (sc != first_sc).sum()
    torch.cuda.synchronize()
    assert int(bad) == 0
    assert ctx.device_status() == binding.SEER_OK


def test_calls_of_different_shapes_interleaved_on_one_context(ctx):
    # different unit counts, block sizes, query-token counts, gate and decode calls share one workspace
    cases = []
    for (B, Hkv, g, b, S, T, seed) in [(1, 8, 5, 64, 8192, 1, 601), (3, 2, 8, 32, 4096, 2, 602), (2, 4, 4, 128, 16384, 3, 603),
                                       (5, 1, 1, 16, 2048, 8, 604)]:
        Hq = g * Hkv
        lens = synth.ragged_lengths(B, S // 2, S, b, seed) - np.int32(seed % 7)       # partial last blocks
        q = synth.normal_bf16((B, T, Hq, 128), seed, "q", DEV)
        k = synth.normal_bf16((B, Hkv, S, 128), seed, "k", DEV)
        v = synth.normal_bf16((B, Hkv, S, 128), seed, "v", DEV)
        n = [-(-int(L) // b) for L in lens]
        keep = [max(1, x // 3) for x in n]
        idx, cnt = synth.random_block_lists(lens, Hkv, b, keep, max(keep), seed, shuffle=True)
        ref = ref_sparse_multi(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.09)
        lens_t = torch.as_tensor(lens, device=DEV)
        cases.append(dict(shape=binding.make_shape(B, Hq, Hkv, 128, b, 0.09), kv=binding.make_kv(k, v, lens_t), q=q, T=T,
                          idx=torch.as_tensor(idx, device=DEV), cnt=torch.as_tensor(cnt, device=DEV), ref=ref,
                          out=torch.empty((B, T, Hq, 128), dtype=torch.bfloat16, device=DEV),
                          lse=torch.empty((B, T, Hq), dtype=torch.float32, device=DEV), keep=(k, v, lens_t)))
    # a gate call of yet another shape in between
    gB, gHkv, gnb = 2, 4, 1500
    sc = synth.normal_f32((gB, gHkv, gnb), 605, "scores", DEV)
    glens = torch.tensor([gnb * 64, 900 * 64], dtype=torch.int32, device=DEV)
    gshape = binding.make_shape(gB, gHkv * 2, gHkv, 128, 64, 0.1)
    ggate = binding.make_gate(128, 1.0e6, None, None, None, gnb)
    gidx = torch.zeros((gB, gHkv, 100), dtype=torch.int32, device=DEV)
    gcnt = torch.zeros((gB, gHkv), dtype=torch.int32, device=DEV)
    want_gidx, want_gcnt = oracle.select(sc.cpu().numpy(), glens.cpu().numpy(), 64, 100 * 64, 100)
    for rep in range(60):
        for c in cases:
            c["out"].fill_(float("nan"))
            ctx.seer_sparse_decode_multi(c["shape"], c["kv"], c["q"], c["T"], c["idx"], c["cnt"], c["idx"].shape[2],
                                         c["out"], c["lse"])
            ctx.seer_gate_select(gshape, ggate, glens, None, sc, 100 * 64, gidx, gcnt, 100)
        if rep % 20 == 19:
            torch.cuda.synchronize()
            for ci, c in enumerate(cases):
                check_attention(c["out"], c["lse"], *c["ref"], what=f"interleaved case {ci} rep {rep}")
            assert np.array_equal(gidx.cpu().numpy(), want_gidx) and np.array_equal(gcnt.cpu().numpy(), want_gcnt)
    assert ctx.device_status() == binding.SEER_OK


def test_a_wait_that_runs_out_is_reported_and_the_context_recovers(ctx):
    # A bounded device-side wait that gives up sets the sticky time-out bit; the status call reports it once,
    # clears the counters a kernel cut short would have left behind, and the context then decodes as before.
    B, Hq, Hkv, d, b, S = 2, 8, 2, 128, 64, 64 * 160
    lens = np.array([S, S - 1000], np.int32)
    q, k, v = make_qkv(B, Hq, Hkv, S, d, 611, DEV)
    n = [-(-int(L) // b) for L in lens]
    idx, cnt = synth.random_block_lists(lens, Hkv, b, [x // 2 for x in n], max(n) // 2, 611)
    ref = oracle.sparse(bits(q), bits(k), bits(v), lens, idx, cnt, b, 0.0884)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.0884)
    lens_t = torch.as_tensor(lens, device=DEV)
    kv = binding.make_kv(k, v, lens_t)
    idx_t, cnt_t = torch.as_tensor(idx, device=DEV), torch.as_tensor(cnt, device=DEV)
    out = torch.empty((B, Hq, d), dtype=torch.bfloat16, device=DEV)
    lse = torch.empty((B, Hq), dtype=torch.float32, device=DEV)

    def decode_and_check(what):
        out.fill_(float("nan"))
        ctx.seer_sparse_decode(shape, kv, q, idx_t, cnt_t, idx.shape[2], out, lse)
        torch.cuda.synchronize()
        check_attention(out, lse, *ref, what=what, strict=True)

    decode_and_check("before")
    assert ctx.device_status() == binding.SEER_OK
    ctx.seer_debug_wait_timeout(1000)                      # a wait on a barrier nobody arrives at, 1000 polls
    torch.cuda.synchronize()
    assert ctx.device_status() == binding.SEER_ERR_TIMEOUT
    assert ctx.device_status() == binding.SEER_OK          # reported once, then clear
    decode_and_check("after the time-out")
    decode_and_check("after the time-out, again")
    assert ctx.device_status() == binding.SEER_OK
