"""Seeded random configurations of the decode entry points against the fp64 oracle: head counts,
block sizes, ragged lengths, list sizes and orders, counts vs padding, paged vs contiguous caches,
one or several query tokens -- many small cases that wander through the corners of the index
arithmetic (partial tiles, units with no work, lists shorter than a tile, pages smaller than blocks)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_08889_b200 import binding, synth
from util import bits, check_attention, to_paged, ref_sparse_multi

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def _draw(case):
    r = synth.np_rng(7000 + case, "config")
    b = int(r.choice([16, 32, 64, 128]))
    Hkv = int(r.choice([1, 2, 3, 8]))
    g = int(r.choice([1, 2, 4, 5, 7, 8]))
    B = int(r.integers(1, 6))
    S = int(r.choice([128, 256, 1024, 4096]))
    S = max(S, b)
    T = int(r.choice([1, 1, 1, 2, 3, 8]))
    lens = r.integers(0, S + 1, size=B).astype(np.int32)
    lens[r.integers(0, B)] = S                                   # at least one full sequence
    if r.random() < 0.3:
        lens[r.integers(0, B)] = int(r.integers(0, 3))           # an empty or nearly empty one
    paged = bool(r.random() < 0.4)
    page_size = int(r.choice([64, 128])) if paged else 0
    frac = float(r.choice([0.1, 0.5, 1.0]))
    use_cnt = bool(r.random() < 0.6)
    dense = bool(r.random() < 0.25)
    return dict(b=b, Hkv=Hkv, g=g, B=B, S=S, T=T, lens=lens, paged=paged, page_size=page_size, frac=frac,
                use_cnt=use_cnt, dense=dense)


@pytest.mark.parametrize("case", range(48))
def test_random_configuration(ctx, case):
    c = _draw(case)
    b, Hkv, g, B, S, T, lens = c["b"], c["Hkv"], c["g"], c["B"], c["S"], c["T"], c["lens"]
    Hq, d, scale = g * Hkv, 128, 0.09
    seed = 7000 + case
    q = synth.normal_bf16((B, T, Hq, d), seed, "q", DEV)
    k = synth.normal_bf16((B, Hkv, S, d), seed, "k", DEV)
    v = synth.normal_bf16((B, Hkv, S, d), seed, "v", DEV)
    n = [-(-int(L) // b) for L in lens]
    keep = [max(1, int(np.ceil(x * c["frac"]))) if x > 0 else 0 for x in n]
    max_sel = max(max(keep), 1) + int(case % 3)
    idx, cnt = synth.random_block_lists(lens, Hkv, b, keep, max_sel, seed, shuffle=bool(case % 2))
    kh, vh = bits(k), bits(v)
    shape = binding.make_shape(B, Hq, Hkv, d, b, scale)
    lens_t = torch.as_tensor(lens, device=DEV)
    if c["paged"] and S % c["page_size"] == 0:
        kp, vp, table = to_paged(k, v, c["page_size"], seed)
        kv = binding.make_kv(kp, vp, lens_t, max_seq_len=S, page_table=table, page_size=c["page_size"])
    else:
        kv = binding.make_kv(k, v, lens_t)
    out = torch.full((B, T, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, T, Hq), float("nan"), dtype=torch.float32, device=DEV)
    if c["dense"]:
        ctx.seer_dense_decode_multi(shape, kv, q, T, out, lse)
        full = np.full((B, Hkv, max(max(n), 1)), -1, np.int32)
        for i in range(B):
            full[i, :, :n[i]] = np.arange(n[i])
        ref = ref_sparse_multi(bits(q), kh, vh, lens, full, None, b, scale)
    else:
        cnt_t = torch.as_tensor(cnt, device=DEV) if c["use_cnt"] else None
        ctx.seer_sparse_decode_multi(shape, kv, q, T, torch.as_tensor(idx, device=DEV), cnt_t, max_sel, out, lse)
        ref = ref_sparse_multi(bits(q), kh, vh, lens, idx, cnt if c["use_cnt"] else None, b, scale)
    torch.cuda.synchronize()
    check_attention(out, lse, *ref, what=f"case {case}: {c}")
    assert ctx.device_status() == binding.SEER_OK


@pytest.mark.parametrize("case", range(24))
def test_random_gate_configuration(ctx, case):
    r = synth.np_rng(9000 + case, "gate-config")
    b = int(r.choice([16, 32, 64, 128]))
    dg = int(r.choice([64, 128, 256]))
    Hkv = int(r.choice([1, 2, 4]))
    g = int(r.choice([1, 2, 4, 5, 8]))
    B = int(r.integers(1, 5))
    nbmax = int(r.choice([3, 40, 511, 512, 513, 1500, 3000]))     # clusters of one to six CTAs
    T = int(r.choice([1, 1, 2, 4, 8]))
    Hq, d, theta = g * Hkv, 128, 1.0e6
    lens = r.integers(0, nbmax * b + 1, size=B).astype(np.int32)
    lens[r.integers(0, B)] = nbmax * b
    seed = 9000 + case
    qn = synth.normal_bf16((B, T, Hq, d), seed, "qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, g * d), seed, "wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nbmax, dg), seed, "kc", DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, theta, wq, None, kc, nbmax)
    lens_t = torch.as_tensor(lens, device=DEV)
    max_sel = int(r.choice([1, 2, 7, 64, nbmax]))
    budget = int(r.choice([0, b, 5 * b, max_sel * b, 10 * nbmax * b]))
    idx = torch.full((B, Hkv, max_sel), 77, dtype=torch.int32, device=DEV)
    cnt = torch.full((B, Hkv), 77, dtype=torch.int32, device=DEV)
    sc = torch.zeros((B, Hkv, nbmax), dtype=torch.float32, device=DEV)
    ctx.seer_gate_select_multi(shape, gate, lens_t, qn, None, T, budget, idx, cnt, max_sel, scores_out=sc)
    torch.cuda.synchronize()
    got_sc = sc.cpu().numpy()
    want_sc = oracle.scores_multi(bits(qn), bits(wq), bits(kc), lens, b, theta)
    for i in range(B):
        jf = min(max(0, int(lens[i]) - T) // b, nbmax)
        if jf:
            assert np.abs(got_sc[i, :, :jf] - want_sc[i, :, :jf]).max() <= 1e-3, (case, i)
    want_idx, want_cnt = oracle.select_multi(got_sc, lens, b, budget, T, max_sel)
    assert np.array_equal(cnt.cpu().numpy(), want_cnt), case
    assert np.array_equal(idx.cpu().numpy(), want_idx), case
    assert ctx.device_status() == binding.SEER_OK
