"""Pins for the AttnGate half of the CPU oracle: K compression (Eq. 1b), rotary
embedding, Q branch and block scores (Eq. 1a, 1c).  No GPU needed.

The checks are special cases that collapse to something a reader can verify by eye
(constant blocks, identity weights, position 0), a restatement of the rotation with
complex numbers, and invariants (norm, relative position, linearity)."""
import os

import numpy as np
import torch

import oracle
from paper_2506_08889_b200 import synth

THETA = 1.0e4


def _bits(t):
    return synth.bf16_bits(t)


def _f64(t):
    return t.to(torch.float64).numpy()


def _rope_complex(y, pos, theta):
    """Rotation written with complex numbers: (y_c + i y_{c+half}) * exp(i pos theta_c)."""
    half = y.shape[0] // 2
    ang = pos * theta ** (-2.0 * np.arange(half) / y.shape[0])
    z = (y[:half] + 1j * y[half:]) * np.exp(1j * ang)
    return np.concatenate([z.real, z.imag])


def test_rope_identity_norm_relative_and_complex_form():
    r = np.random.default_rng(0)
    x, y = r.normal(size=32), r.normal(size=32)
    assert np.array_equal(oracle.rope(x, 0, THETA), x)
    for pos in (1, 63, 4096, 131071):
        rx = oracle.rope(x, pos, THETA)
        assert abs(np.linalg.norm(rx) - np.linalg.norm(x)) < 1e-12
        assert np.allclose(rx, _rope_complex(x, pos, THETA), atol=1e-12)
    # <R_m x, R_n y> depends on m - n only
    a = oracle.rope(x, 1000, THETA) @ oracle.rope(y, 936, THETA)
    b = oracle.rope(x, 64, THETA) @ oracle.rope(y, 0, THETA)
    assert abs(a - b) < 1e-10
    # first pair rotates by exactly pos radians (theta^0 = 1): a quarter turn maps (1,0)->(0,1)
    e = np.zeros(8); e[0] = 1.0
    out = oracle.rope(e, np.pi / 2, THETA)
    assert abs(out[0]) < 1e-15 and abs(out[4] - 1.0) < 1e-15
    # the last pair turns slowest: angle = pos * theta^(-(dg-2)/dg)
    e = np.zeros(8); e[3] = 1.0
    out = oracle.rope(e, 10.0, THETA)
    ang = 10.0 * THETA ** (-6.0 / 8.0)
    assert abs(out[3] - np.cos(ang)) < 1e-15 and abs(out[7] - np.sin(ang)) < 1e-15


def test_memory_ratio_golden_fixture():
    # the paper states the size of the K compression cache relative to the KV cache
    path = os.path.join(os.path.dirname(__file__), "golden", "kcomp_cache_ratio.txt")
    vals = {}
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            key, val = line.split("=")
            vals[key.strip()] = val.strip()
    b, d = int(vals["block_size"]), 128
    dg = d
    kc_bytes_per_block = dg * 2
    kv_bytes_per_block = 2 * b * d * 2
    num, den = vals["kcomp_over_kv"].split("/")
    assert kc_bytes_per_block * int(den) == kv_bytes_per_block * int(num)
    # and the oracle's output really has that shape: one dg vector per (head, block)
    k = synth.normal_bf16((1, 2, 2 * b, d), 1, "k")
    w = synth.normal_bf16((2, dg, 3 * d), 1, "w", std=0.02)
    kc, _ = oracle.kcomp(_bits(k), _bits(w), b, 0, 2, 2, THETA)
    assert kc.shape == (1, 2, 2, dg) and kc.nbytes * int(den) == 2 * k.numel() * 2 * int(num)


def test_kcomp_constant_block_with_selector_weights():
    B, Hkv, d, dg, b = 1, 2, 16, 16, 8
    rows = synth.normal_bf16((B, Hkv, 3, 1, d), 2, "rows")
    k = rows.expand(B, Hkv, 3, b, d).reshape(B, Hkv, 3 * b, d).contiguous()   # each block constant
    eye = torch.eye(d, dtype=torch.bfloat16)
    zero = torch.zeros(d, d, dtype=torch.bfloat16)
    for which in range(3):                       # [I 0 0], [0 I 0], [0 0 I]
        blocks = [zero, zero, zero]
        blocks[which] = eye
        w = torch.cat(blocks, dim=1).unsqueeze(0).repeat(Hkv, 1, 1)
        kc, kc64 = oracle.kcomp(_bits(k), _bits(w), b, 0, 3, 3, THETA)
        for h in range(Hkv):
            for j in range(3):
                want = _rope_complex(_f64(rows[0, h, j, 0]), j * b, THETA)
                assert np.allclose(kc64[0, h, j], want, atol=1e-13)
                if j == 0:                      # position 0: rotation is the identity
                    assert np.array_equal(kc[0, h, 0], _bits(rows[0, h, 0, 0]))


def test_kcomp_pools_max_min_avg_in_that_order():
    B, Hkv, d, dg, b = 1, 1, 4, 12, 4
    k = torch.tensor([[[[1, -1, 2, 0], [3, 1, -2, 0], [-5, -1, 2, 8], [1, 1, -2, 0]]]],
                     dtype=torch.bfloat16)
    # alternating +-1 in channel 1 -> avg 0; channel 2 alternating +-2 -> avg 0
    w = torch.eye(12, dtype=torch.bfloat16).unsqueeze(0)     # dg = 3d: output = features
    kc, kc64 = oracle.kcomp(_bits(k), _bits(w), b, 0, 1, 1, THETA)
    want = np.array([3, 1, 2, 8, -5, -1, -2, 0, 0, 0, 0, 2], dtype=np.float64)
    assert np.array_equal(kc64[0, 0, 0], want)


def test_kcomp_general_case_against_numpy_restatement():
    B, Hkv, d, dg, b, nb = 2, 2, 16, 8, 8, 5
    k = synth.normal_bf16((B, Hkv, nb * b, d), 3, "k")
    w = synth.normal_bf16((Hkv, dg, 3 * d), 3, "w", std=0.1)
    kc, kc64 = oracle.kcomp(_bits(k), _bits(w), b, 1, 3, nb, THETA)
    kk, ww = _f64(k), _f64(w)
    for i in range(B):
        for h in range(Hkv):
            for j in range(nb):
                if not (1 <= j < 4):
                    assert np.all(kc[i, h, j] == 0)      # outside the range: untouched
                    continue
                blk = kk[i, h, j * b:(j + 1) * b]
                feat = np.concatenate([blk.max(0), blk.min(0), blk.mean(0)])
                want = _rope_complex(ww[h] @ feat, j * b, THETA)
                assert np.allclose(kc64[i, h, j], want, atol=1e-12)
                got = _f64(synth.bits_to_bf16(kc[i, h, j]))
                assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 1e-30)


def test_scores_reduce_to_plain_dot_product():
    B, Hq, Hkv, d, nb = 1, 6, 2, 16, 7
    g, dg = 3, 16
    qn = synth.normal_bf16((B, Hq, d), 4, "qn")
    kc = synth.normal_bf16((B, Hkv, nb, dg), 4, "kc")
    for u in range(g):                           # W_q picks the u-th head of each group
        w = torch.zeros(Hkv, dg, g * d, dtype=torch.bfloat16)
        w[:, :, u * d:(u + 1) * d] = torch.eye(d, dtype=torch.bfloat16)
        sc, qg = oracle.scores(_bits(qn), _bits(w), _bits(kc), [nb], [0], THETA)
        for h in range(Hkv):
            assert np.array_equal(qg[0, h], _f64(qn[0, h * g + u]))
            want = _f64(kc[0, h]) @ _f64(qn[0, h * g + u]) / np.sqrt(dg)
            assert np.allclose(sc[0, h], want, atol=1e-13)


def test_scores_general_linearity_and_entry_limit():
    B, Hq, Hkv, d, dg, nb = 2, 4, 2, 8, 8, 6
    g = 2
    qn = synth.normal_bf16((B, Hq, d), 5, "qn")
    w = synth.normal_bf16((Hkv, dg, g * d), 5, "w", std=0.2)
    kc = synth.normal_bf16((B, Hkv, nb, dg), 5, "kc")
    n_entries, qpos = [6, 4], [383, 300]
    sc, qg = oracle.scores(_bits(qn), _bits(w), _bits(kc), n_entries, qpos, THETA)
    for i in range(B):
        for h in range(Hkv):
            x = _f64(qn[i, h * g:(h + 1) * g]).reshape(-1)        # head-major concat
            want_q = _rope_complex(_f64(w[h]) @ x, qpos[i], THETA)
            assert np.allclose(qg[i, h], want_q, atol=1e-12)
            want = _f64(kc[i, h, :n_entries[i]]) @ want_q / np.sqrt(dg)
            assert np.allclose(sc[i, h, :n_entries[i]], want, atol=1e-12)
            assert np.all(sc[i, h, n_entries[i]:] == 0.0)
    # doubling Q_nope (exact in bf16) doubles every score
    sc2, _ = oracle.scores(_bits(qn * 2), _bits(w), _bits(kc), n_entries, qpos, THETA)
    assert np.allclose(sc2, 2 * sc, atol=1e-12)


def test_score_depends_on_relative_position_only():
    # one gate query against a compressed key built by the K branch: shifting both
    # positions by the same number of blocks leaves the score unchanged (up to the bf16
    # rounding of the cached entry, which is why the f64 entries are compared)
    B, Hkv, d, dg, b = 1, 1, 8, 8, 4
    row = synth.normal_bf16((d,), 6, "row")
    k = row.expand(1, 1, 6 * b, d).contiguous()
    wk = torch.cat([torch.eye(d), torch.zeros(d, 2 * d)], dim=1).to(torch.bfloat16).unsqueeze(0)
    _, kc64 = oracle.kcomp(_bits(k), _bits(wk), b, 0, 6, 6, THETA)
    x = np.random.default_rng(1).normal(size=dg)
    s1 = oracle.rope(x, 2 * b + 3, THETA) @ kc64[0, 0, 1]
    s2 = oracle.rope(x, 5 * b + 3, THETA) @ kc64[0, 0, 4]
    assert abs(s1 - s2) < 1e-10


# ---- gate scores for several query tokens ---------------------------------------------------------

def test_multi_token_scores_are_the_maximum_of_single_token_scores_at_each_tokens_position():
    B, T, Hq, Hkv, d, dg, nb, b = 2, 3, 4, 2, 8, 8, 9, 16
    qn = synth.normal_bf16((B, T, Hq, d), 6, "qn")
    w = synth.normal_bf16((Hkv, dg, 2 * d), 6, "w", std=0.2)
    kc = synth.normal_bf16((B, Hkv, nb, dg), 6, "kc")
    lens = np.array([9 * 16, 5 * 16 + 2], np.int32)     # 82: the three tokens straddle blocks 4 and 5
    got = oracle.scores_multi(_bits(qn), _bits(w), _bits(kc), lens, b, THETA)
    jf = [(int(L) - T) // b for L in lens]
    assert jf == [8, 4]
    per_token = []
    for t in range(T):
        sc, _ = oracle.scores(_bits(qn[:, t]), _bits(w), _bits(kc), jf, [int(L) - T + t for L in lens], THETA)
        per_token.append(sc)
    want = np.max(np.stack(per_token), axis=0)
    for i in range(B):
        assert np.allclose(got[i, :, :jf[i]], want[i, :, :jf[i]], rtol=0, atol=1e-13)
        assert np.all(got[i, :, jf[i]:] == 0.0)
    # a single token: the single-token routine itself
    one = oracle.scores_multi(_bits(qn[:, :1]), _bits(w), _bits(kc), lens, b, THETA)
    ref, _ = oracle.scores(_bits(qn[:, 0]), _bits(w), _bits(kc), [(int(L) - 1) // b for L in lens],
                           [int(L) - 1 for L in lens], THETA)
    assert np.array_equal(one, ref)
