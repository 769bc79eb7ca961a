"""Pins for the attention half of the CPU oracle (no GPU needed).

Each test checks ``oracle.dense`` / ``oracle.sparse`` against something the mathematics
fixes independently of the oracle's own code: closed forms, a library routine, a second
formulation (streaming softmax over arbitrary partitions merged by log-sum-exp, which is
the identity the split-KV combine relies on), and invariances.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_08889_b200 import synth


def _bits(t):
    return synth.bf16_bits(t)


def _f64(t):
    return t.to(torch.float64).numpy()


def _mk(B, Hq, Hkv, S, d, seed, name="t"):
    q = synth.normal_bf16((B, Hq, d), seed, name + "q")
    k = synth.normal_bf16((B, Hkv, S, d), seed, name + "k")
    v = synth.normal_bf16((B, Hkv, S, d), seed, name + "v")
    return q, k, v


def test_bf16_rounding_helper_ties_to_even_and_specials():
    # exhaustive over all finite bf16 values: exact values round to themselves,
    # midpoints go to the even neighbour
    bits = np.arange(0, 0x7f80, dtype=np.uint16)
    vals = synth.bits_to_bf16(bits).to(torch.float64).numpy()
    for i in list(range(0, 300)) + list(range(0x3f00, 0x4100)) + list(range(0x7f00, 0x7f7f)):
        assert oracle.round_bf16(vals[i]) == bits[i]
        assert oracle.round_bf16(-vals[i]) == (bits[i] | 0x8000)
        mid = 0.5 * (vals[i] + vals[i + 1])
        want = bits[i] if bits[i] % 2 == 0 else bits[i + 1]
        assert oracle.round_bf16(mid) == want, hex(i)
        assert oracle.round_bf16(np.nextafter(mid, np.inf)) == bits[i + 1]
        assert oracle.round_bf16(np.nextafter(mid, -np.inf)) == bits[i]
    assert oracle.round_bf16(float("inf")) == 0x7f80
    assert oracle.round_bf16(1e39) == 0x7f80
    # agrees with torch's own float32 -> bf16 rounding on random float32 values
    x = torch.randn(4096, generator=torch.Generator().manual_seed(3), dtype=torch.float32)
    want = synth.bf16_bits(x.to(torch.bfloat16))
    got = np.array([oracle.round_bf16(float(t)) for t in x], dtype=np.uint16)
    assert np.array_equal(got, want)


def test_single_token_is_its_value_row():
    q, k, v = _mk(2, 4, 2, 1, 16, 1)
    out, lse = oracle.dense(_bits(q), _bits(k), _bits(v), [1, 1], 0.3)
    for i in range(2):
        for hq in range(4):
            h = hq // 2
            assert np.allclose(out[i, hq], _f64(v[i, h, 0]), rtol=0, atol=1e-15)
            want = 0.3 * float(_f64(q[i, hq]) @ _f64(k[i, h, 0]))
            assert abs(lse[i, hq] - want) < 1e-12


def test_equal_keys_give_mean_of_values():
    q, k, v = _mk(1, 4, 1, 37, 32, 2)
    k[:] = k[:, :, :1]
    out, lse = oracle.dense(_bits(q), _bits(k), _bits(v), [37], 0.25)
    mean_v = _f64(v[0, 0]).mean(axis=0)
    for hq in range(4):
        assert np.allclose(out[0, hq], mean_v, atol=1e-13)
        s = 0.25 * float(_f64(q[0, hq]) @ _f64(k[0, 0, 0]))
        assert abs(lse[0, hq] - (s + np.log(37.0))) < 1e-12


def test_dominant_key_selects_its_row():
    d = 16
    q = torch.zeros(1, 1, d, dtype=torch.bfloat16); q[0, 0, 0] = 8.0
    k = torch.zeros(1, 1, 20, d, dtype=torch.bfloat16); k[0, 0, 7, 0] = 16.0   # score 128 vs 0
    v = synth.normal_bf16((1, 1, 20, d), 3, "v")
    out, lse = oracle.dense(_bits(q), _bits(k), _bits(v), [20], 1.0)
    assert np.allclose(out[0, 0], _f64(v[0, 0, 7]), atol=1e-12)
    assert abs(lse[0, 0] - 128.0) < 1e-12


def test_dense_matches_torch_fp64_attention_gqa_and_ragged():
    B, Hq, Hkv, S, d = 3, 6, 2, 50, 24
    q, k, v = _mk(B, Hq, Hkv, S, d, 4)
    lens = [50, 17, 1]
    scale = 0.17
    out, lse = oracle.dense(_bits(q), _bits(k), _bits(v), lens, scale)
    g = Hq // Hkv
    for i in range(B):
        L = lens[i]
        qq = q[i].to(torch.float64).unsqueeze(1)                       # [Hq,1,d]
        kk = k[i, :, :L].to(torch.float64).repeat_interleave(g, dim=0)  # [Hq,L,d]
        vv = v[i, :, :L].to(torch.float64).repeat_interleave(g, dim=0)
        ref = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv, scale=scale)
        assert np.allclose(out[i], ref[:, 0].numpy(), atol=1e-12)
        s = (qq @ kk.transpose(1, 2))[:, 0] * scale
        assert np.allclose(lse[i], torch.logsumexp(s, dim=-1).numpy(), atol=1e-12)


def test_strided_token_major_layout_gives_same_result():
    B, Hq, Hkv, S, d = 2, 4, 2, 33, 16
    q, k, v = _mk(B, Hq, Hkv, S, d, 5)
    lens = [33, 20]
    ref = oracle.dense(_bits(q), _bits(k), _bits(v), lens, 0.2)
    k2 = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)       # [B,S,Hkv,d] storage
    v2 = v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert not k2.is_contiguous()
    got = oracle.dense(_bits(q), _bits(k2), _bits(v2), lens, 0.2)
    assert np.array_equal(ref[0], got[0]) and np.array_equal(ref[1], got[1])


def test_full_selection_equals_dense():
    B, Hq, Hkv, S, d, b = 2, 8, 2, 200, 32, 16
    q, k, v = _mk(B, Hq, Hkv, S, d, 6)
    lens = np.array([200, 93], np.int32)          # 93: partial last block
    max_sel = 13
    idx = np.full((B, Hkv, max_sel), -1, np.int32)
    cnt = np.zeros((B, Hkv), np.int32)
    for i in range(B):
        n = -(-int(lens[i]) // b)
        idx[i, :, :n] = np.arange(n)
        cnt[i] = n
    d_out, d_lse = oracle.dense(_bits(q), _bits(k), _bits(v), lens, 0.11)
    s_out, s_lse = oracle.sparse(_bits(q), _bits(k), _bits(v), lens, idx, cnt, b, 0.11)
    assert np.allclose(d_out, s_out, atol=1e-14) and np.allclose(d_lse, s_lse, atol=1e-13)
    # block_cnt omitted: the -1 padding is skipped
    s_out2, s_lse2 = oracle.sparse(_bits(q), _bits(k), _bits(v), lens, idx, None, b, 0.11)
    assert np.array_equal(s_out, s_out2) and np.array_equal(s_lse, s_lse2)


def _streaming_reference(qv, kk, vv, token_groups, scale):
    """Independent formulation: online softmax per token group, then LSE merge."""
    parts = []
    for toks in token_groups:
        m, l, acc = -np.inf, 0.0, np.zeros(vv.shape[1])
        for t in toks:
            s = scale * float(qv @ kk[t])
            m_new = max(m, s)
            corr = np.exp(m - m_new) if np.isfinite(m) else 0.0
            p = np.exp(s - m_new)
            l = l * corr + p
            acc = acc * corr + p * vv[t]
            m = m_new
        if toks:
            parts.append((acc / l, m + np.log(l)))
    lses = np.array([p[1] for p in parts])
    lse = np.log(np.sum(np.exp(lses - lses.max()))) + lses.max()
    o = sum(np.exp(p[1] - lse) * p[0] for p in parts)
    return o, lse


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_sparse_matches_streaming_partitioned_bruteforce(seed):
    B, Hq, Hkv, d, b = 2, 6, 2, 16, 8
    r = np.random.default_rng(seed)
    lens = np.array([77, 64], np.int32)
    q, k, v = _mk(B, Hq, Hkv, 80, d, seed)
    idx, cnt = synth.random_block_lists(lens, Hkv, b, [5, 3], 9, seed, shuffle=True)
    scale = 0.3
    out, lse = oracle.sparse(_bits(q), _bits(k), _bits(v), lens, idx, cnt, b, scale)
    g = Hq // Hkv
    for i in range(B):
        for hq in range(Hq):
            h = hq // g
            toks = []
            for j in idx[i, h, :cnt[i, h]]:
                toks += [t for t in range(j * b, (j + 1) * b) if t < lens[i]]
            r.shuffle(toks)
            cuts = sorted(r.choice(np.arange(1, len(toks)), size=3, replace=False))
            groups = [toks[a:c] for a, c in zip([0] + cuts, cuts + [len(toks)])]
            o, l = _streaming_reference(_f64(q[i, hq]), _f64(k[i, h]), _f64(v[i, h]), groups, scale)
            assert np.allclose(out[i, hq], o, atol=1e-12)
            assert abs(lse[i, hq] - l) < 1e-12


def test_sparse_invariances_permutation_padding_duplicates_out_of_range():
    B, Hq, Hkv, d, b = 1, 4, 2, 16, 8
    lens = np.array([60], np.int32)               # 8 blocks, last one partial (4 tokens)
    q, k, v = _mk(B, Hq, Hkv, 64, d, 21)
    idx = np.array([[[1, 4, 7, -1, -1, -1], [0, 2, 7, -1, -1, -1]]], np.int32)
    cnt = np.array([[3, 3]], np.int32)
    ref = oracle.sparse(_bits(q), _bits(k), _bits(v), lens, idx, cnt, b, 0.2)
    perm = np.array([[[7, 1, 4, -1, -1, -1], [2, 7, 0, -1, -1, -1]]], np.int32)
    got = oracle.sparse(_bits(q), _bits(k), _bits(v), lens, perm, cnt, b, 0.2)
    assert np.allclose(ref[0], got[0], atol=1e-14)
    # -1 in the middle, duplicates and out-of-range entries are all ignored
    junk = np.array([[[1, -1, 4, 7, 4, 8], [99, 0, 2, 7, 7, -1]]], np.int32)
    got = oracle.sparse(_bits(q), _bits(k), _bits(v), lens, junk, None, b, 0.2)
    assert np.allclose(ref[0], got[0], atol=1e-14) and np.allclose(ref[1], got[1], atol=1e-14)
    # tokens past the length never contribute: change them and nothing moves
    k2, v2 = k.clone(), v.clone()
    k2[:, :, 60:] = 50.0
    v2[:, :, 60:] = -77.0
    got = oracle.sparse(_bits(q), _bits(k2), _bits(v2), lens, idx, cnt, b, 0.2)
    assert np.array_equal(ref[0], got[0]) and np.array_equal(ref[1], got[1])


def test_empty_selection_gives_zero_and_minus_inf():
    q, k, v = _mk(1, 2, 1, 16, 8, 22)
    idx = np.full((1, 1, 4), -1, np.int32)
    out, lse = oracle.sparse(_bits(q), _bits(k), _bits(v), [16], idx, np.zeros((1, 1), np.int32), 8, 1.0)
    assert np.all(out == 0.0) and np.all(np.isneginf(lse))


def test_key_shift_moves_lse_only():
    # adding one vector c to every key shifts every score by scale*<q,c>
    B, Hq, Hkv, S, d = 1, 2, 1, 40, 8
    q = synth.bits_to_bf16(synth.bf16_bits(synth.normal_bf16((B, Hq, d), 31, "q")))
    # small integers are exact in bf16, so k + c is exact too
    r = np.random.default_rng(5)
    k = torch.tensor(r.integers(-3, 4, size=(B, Hkv, S, d)), dtype=torch.bfloat16)
    c = torch.tensor(r.integers(-2, 3, size=(d,)), dtype=torch.bfloat16)
    v = synth.normal_bf16((B, Hkv, S, d), 31, "v")
    o1, l1 = oracle.dense(_bits(q), _bits(k), _bits(v), [S], 0.5)
    o2, l2 = oracle.dense(_bits(q), _bits(k + c), _bits(v), [S], 0.5)
    assert np.allclose(o1, o2, atol=1e-13)
    for hq in range(Hq):
        assert abs((l2[0, hq] - l1[0, hq]) - 0.5 * float(_f64(q[0, hq]) @ _f64(c))) < 1e-12


def test_transposed_operand_or_wrong_group_mapping_would_be_caught():
    # distinct K and V, g = 3 and Hkv = 2: query head 3 must read KV head 1, not 0 or 3 % 2
    B, Hq, Hkv, S, d = 1, 6, 2, 9, 8
    q, k, v = _mk(B, Hq, Hkv, S, d, 41)
    out, _ = oracle.dense(_bits(q), _bits(k), _bits(v), [S], 0.4)
    for hq, h in [(2, 0), (3, 1), (5, 1)]:
        s = 0.4 * (_f64(k[0, h]) @ _f64(q[0, hq]))
        p = np.exp(s - s.max()); p /= p.sum()
        assert np.allclose(out[0, hq], p @ _f64(v[0, h]), atol=1e-13)


# ---- T query tokens per sequence (the query-level parallelism Sec. 6 points to) ------------------

def _mk_multi(B, T, Hq, Hkv, S, d, seed, name="m"):
    q = synth.normal_bf16((B, T, Hq, d), seed, name + "q")
    k = synth.normal_bf16((B, Hkv, S, d), seed, name + "k")
    v = synth.normal_bf16((B, Hkv, S, d), seed, name + "v")
    return q, k, v


def test_multi_token_with_one_token_is_the_single_token_routine():
    q, k, v = _mk_multi(2, 1, 4, 2, 50, 16, 31)
    lens = [50, 37]
    idx = np.array([[[0, 3, 6], [1, 2, 6]], [[4, 0, -1], [2, 4, 1]]], np.int32)
    cnt = np.array([[3, 3], [2, 3]], np.int32)
    out, lse = oracle.sparse_multi(_bits(q), _bits(k), _bits(v), lens, idx, cnt, 8, 0.25)
    want, want_lse = oracle.sparse(_bits(q[:, 0]), _bits(k), _bits(v), lens, idx, cnt, 8, 0.25)
    assert np.array_equal(out[:, 0], want) and np.array_equal(lse[:, 0], want_lse)


@pytest.mark.parametrize("T", [2, 3, 8])
def test_multi_token_query_t_is_single_token_decode_on_the_cache_cut_after_its_position(T):
    # query t at position L-T+t sees exactly what a one-token decode sees when the cache ends there
    B, Hq, Hkv, S, d, b = 2, 6, 2, 70, 16, 8
    q, k, v = _mk_multi(B, T, Hq, Hkv, S, d, 32 + T)
    lens = np.array([70, 41], np.int32)          # 41: the T tokens straddle a block boundary for T >= 2
    rng = synth.np_rng(5, "multi-lists")
    idx = np.stack([np.stack([rng.permutation(9)[:6] for _ in range(Hkv)]) for _ in range(B)]).astype(np.int32)
    idx[:, :, 0] = (lens[:, None] - 1) // b      # the last block is always there
    idx[0, 0, 1] = (70 - T) // b                 # and, for one unit, the block the first new token is in
    out, lse = oracle.sparse_multi(_bits(q), _bits(k), _bits(v), lens, idx, None, b, 0.3)
    for t in range(T):
        cut = lens - T + t + 1
        want, want_lse = oracle.sparse(_bits(q[:, t]), _bits(k), _bits(v), cut, idx, None, b, 0.3)
        assert np.allclose(out[:, t], want, rtol=0, atol=1e-14)
        assert np.allclose(lse[:, t], want_lse, rtol=0, atol=1e-13)


def test_multi_token_matches_masked_softmax_written_with_matrices():
    # brute force: one [T, L] mask (listed blocks AND causal) and a plain softmax in numpy
    B, T, Hq, Hkv, S, d, b = 1, 4, 4, 2, 30, 8, 4
    q, k, v = _mk_multi(B, T, Hq, Hkv, S, d, 40)
    L = 27
    idx = np.array([[[6, 1, 4, 5], [6, 0, 2, 3]]], np.int32)
    out, lse = oracle.sparse_multi(_bits(q), _bits(k), _bits(v), [L], idx, None, b, 0.5)
    pos = np.arange(L)
    for hq in range(Hq):
        h = hq // 2
        in_list = np.isin(pos // b, idx[0, h])
        qpos = L - T + np.arange(T)
        mask = in_list[None, :] & (pos[None, :] <= qpos[:, None])
        s = 0.5 * _f64(q[0, :, hq]) @ _f64(k[0, h, :L]).T
        s = np.where(mask, s, -np.inf)
        w = np.exp(s - s.max(axis=1, keepdims=True))
        z = w.sum(axis=1, keepdims=True)
        assert np.allclose(out[0, :, hq], (w / z) @ _f64(v[0, h, :L]), rtol=0, atol=1e-14)
        assert np.allclose(lse[0, :, hq], s.max(axis=1) + np.log(z[:, 0]), rtol=0, atol=1e-13)


def test_multi_token_earlier_queries_do_not_see_later_tokens_and_unseen_rows_are_zero():
    B, T, Hq, Hkv, S, d, b = 1, 3, 2, 1, 24, 8, 8
    q, k, v = _mk_multi(B, T, Hq, Hkv, S, d, 41)
    L = 17                                        # block 2 holds position 16 only
    idx = np.array([[[2, 0]]], np.int32)
    out, lse = oracle.sparse_multi(_bits(q), _bits(k), _bits(v), [L], idx, None, b, 0.4)
    k2, v2 = k.clone(), v.clone()
    k2[0, 0, 16] += 1.0                           # the last token: visible to query 2 only
    v2[0, 0, 16] -= 2.0
    out2, lse2 = oracle.sparse_multi(_bits(q), _bits(k2), _bits(v2), [L], idx, None, b, 0.4)
    assert np.array_equal(out[0, :2], out2[0, :2]) and np.array_equal(lse[0, :2], lse2[0, :2])
    assert not np.allclose(out[0, 2], out2[0, 2])
    # only the last block listed: queries 0 and 1 (positions 14, 15) see nothing at all
    out3, lse3 = oracle.sparse_multi(_bits(q), _bits(k), _bits(v), [L], np.array([[[2]]], np.int32), None, b, 0.4)
    assert np.all(out3[0, :2] == 0.0) and np.all(np.isneginf(lse3[0, :2]))
    assert np.allclose(out3[0, 2], _f64(v[0, 0, 16])[None, :], rtol=0, atol=1e-15)
