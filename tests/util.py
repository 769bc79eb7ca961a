"""Shared helpers of the GPU parity tests: run the library through its C ABI on seeded inputs
and the fp64 oracle on host copies of the same bits, and compare within the stated bounds."""
import numpy as np
import torch

import oracle
from paper_2506_08889_b200 import synth

# attention parity bounds (bf16 inputs, fp32 accumulation, bf16 output) against the fp64 oracle
MAX_ABS = 2e-3
REL_L2 = 5e-3


def bits(t):
    return synth.bf16_bits(t)


def _abs_bits(v):
    """bf16 bit patterns of |v| (sign bit cleared)."""
    return np.asarray(v) & np.uint16(0x7FFF)


def ref_sparse(q, k, v, lens, idx, cnt, b, scale):
    """oracle.sparse plus the weight of the values behind every output element,
    a[i,h,c] = sum_t p_t |v[t,c]| (the oracle run once more on |V|): (out, lse, a)."""
    o, l = oracle.sparse(q, k, v, lens, idx, cnt, b, scale)
    a, _ = oracle.sparse(q, k, _abs_bits(v), lens, idx, cnt, b, scale)
    return o, l, a


def ref_dense(q, k, v, lens, scale):
    o, l = oracle.dense(q, k, v, lens, scale)
    a, _ = oracle.dense(q, k, _abs_bits(v), lens, scale)
    return o, l, a


def ref_sparse_multi(q, k, v, lens, idx, cnt, b, scale):
    o, l = oracle.sparse_multi(q, k, v, lens, idx, cnt, b, scale)
    a, _ = oracle.sparse_multi(q, k, _abs_bits(v), lens, idx, cnt, b, scale)
    return o, l, a


def check_attention(out_gpu, lse_gpu, out_ref, lse_ref, pabsv=None, what="", strict=False):
    """strict: max abs error <= 2e-3 outright (the bound stated for the long-context
    workloads, whose outputs are averages over thousands of tokens and stay well below 1).
    Otherwise (short or degenerate sequences, |o| of order 1) the same bound plus the two terms
    that no bf16 pipeline can avoid, each taken from the data of the element itself.  bf16 keeps 8
    significant bits, so rounding to nearest moves a value by at most half a spacing, which is at
    most 2^-8 of the value.  (1) The bf16 output: half the bf16 spacing at |o|.  (2) The
    probabilities are rounded to bf16 before P.V while the normalising sum keeps them in fp32: at
    most 2^-8 sum_t p_t |v_t,c| -- `pabsv`, which the ref_* helpers above compute with the oracle
    on |V|.  The relative L2 bound is 5e-3 in both modes."""
    got = out_gpu.detach().to(torch.float64).cpu().numpy()
    diff = np.abs(got - out_ref)
    err = diff.max() if diff.size else 0.0
    rel = np.linalg.norm(got - out_ref) / max(np.linalg.norm(out_ref), 1e-30)
    if strict:
        assert err <= MAX_ABS, f"{what}: max abs err {err}"
    else:
        assert pabsv is not None, "the non-strict bound needs sum_t p_t |v_t| (use the ref_* helpers)"
        bound = MAX_ABS + 0.5 * bf16_ulp(out_ref) + 2.0 ** -8 * pabsv
        excess = (diff - bound).max() if diff.size else 0.0
        assert excess <= 0, f"{what}: abs err exceeds 2e-3 + ulp(ref)/2 + 2^-8 sum p|v| by {excess} (max abs err {err})"
    assert rel <= REL_L2, f"{what}: rel L2 err {rel}"
    if lse_gpu is not None:
        lg = lse_gpu.detach().to(torch.float64).cpu().numpy()
        fin = np.isfinite(lse_ref)
        assert np.array_equal(np.isneginf(lg), np.isneginf(lse_ref)), f"{what}: -inf pattern of lse"
        if fin.any():
            lerr = np.abs(lg[fin] - lse_ref[fin]).max()
            assert lerr <= 2e-3, f"{what}: lse err {lerr}"
    return err, rel


def bf16_ulp(x):
    """Spacing of bf16 numbers at |x|: 2^(floor(log2|x|) - 7) (0 for x == 0)."""
    ax = np.abs(np.asarray(x, np.float64))
    e = np.floor(np.log2(np.where(ax > 0, ax, 1.0)))
    return np.where(ax > 0, 2.0 ** (e - 7), 0.0)


def kc_tolerance(want_f64):
    """Bound on |Kc_gpu - Kc_oracle| per entry: one bf16 ulp at the fp64 value, plus the fp32-vs-fp64
    accumulation noise over the 384-term projection, which is what is left for entries near zero."""
    want_f64 = np.asarray(want_f64)
    return bf16_ulp(want_f64) + 1e-5 * np.abs(want_f64).max()


def make_qkv(B, Hq, Hkv, S, d, seed, device, name="", token_major=False):
    q = synth.normal_bf16((B, Hq, d), seed, name + "q", device)
    if token_major:
        k = synth.normal_bf16((B, S, Hkv, d), seed, name + "k", device).permute(0, 2, 1, 3)
        v = synth.normal_bf16((B, S, Hkv, d), seed, name + "v", device).permute(0, 2, 1, 3)
    else:
        k = synth.normal_bf16((B, Hkv, S, d), seed, name + "k", device)
        v = synth.normal_bf16((B, Hkv, S, d), seed, name + "v", device)
    return q, k, v


def to_paged(k, v, page_size, seed):
    """Scatter a [B,Hkv,S,d] cache into a pool [pages,Hkv,P,d] under a random page permutation."""
    B, Hkv, S, d = k.shape
    assert S % page_size == 0
    ppb = S // page_size
    n_pages = B * ppb + 3                       # a few spare pages that stay unused
    perm = synth.page_permutation(n_pages, seed)
    table = torch.from_numpy(perm[: B * ppb].reshape(B, ppb).copy()).to(k.device)
    kp = torch.zeros((n_pages, Hkv, page_size, d), dtype=k.dtype, device=k.device)
    vp = torch.zeros_like(kp)
    kb = k.reshape(B, Hkv, ppb, page_size, d).permute(0, 2, 1, 3, 4).reshape(B * ppb, Hkv, page_size, d)
    vb = v.reshape(B, Hkv, ppb, page_size, d).permute(0, 2, 1, 3, 4).reshape(B * ppb, Hkv, page_size, d)
    kp[table.reshape(-1).long()] = kb
    vp[table.reshape(-1).long()] = vb
    return kp, vp, table.to(torch.int32).contiguous()
