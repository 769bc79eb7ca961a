"""seer_gate_select_static: gate scoring + selection for callers that may not allocate.

A serving process that gives all of its HBM to its own pool at start-up, or code running where
the CUDA allocator must not be entered, cannot create a context (seer_create allocates the
workspace).  For them the library keeps the gate's scratch in a fixed array of its own image.

The array is only used when a unit has more compressed keys than the one-kernel gate holds in
shared memory (more than 8192): the gate then runs as two kernels that pass the gate query, the
scores and per-unit tickets through it.  The first test below takes that path, twice in a row with
different inputs (once with the scores going to the caller, once with the scores staying in the
array), and checks each call against the fp64 oracle and against the ordinary context-based
seer_gate_select: scores within the tolerance the gate tests use, the selected block lists exactly.
The second call finds the first call's query, scores and (re-armed) tickets in the array and must not
be misled by them.  The second test does the same for a size that takes the one-kernel path.

The file name makes pytest collect it last, so a run that stops at the first failure has
already been through every other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_08889_b200 import binding, synth
from util import bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
THETA = 1.0e6


def _inputs(seed, B, Hq, Hkv, d, dg, nbmax):
    g = Hq // Hkv
    qn = synth.normal_bf16((B, Hq, d), seed, "zz:qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, g * d), seed, "zz:wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nbmax, dg), seed, "zz:kc", DEV)
    return qn, wq, kc


def _two_calls(B, Hq, Hkv, dg, b, nbmax, lens, max_sel, seeds):
    d = 128
    lens_t = torch.as_tensor(lens, device=DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    budget = max_sel * b
    n = [-(-int(L) // b) for L in lens]
    ctx = binding.Context(0)
    try:
        for call, seed in enumerate(seeds):
            qn, wq, kc = _inputs(seed, B, Hq, Hkv, d, dg, nbmax)
            gate = binding.make_gate(dg, THETA, wq, None, kc, nbmax)
            # the context-based entry point on the same inputs
            ctx_idx = torch.full((B, Hkv, max_sel), 7, dtype=torch.int32, device=DEV)
            ctx_cnt = torch.full((B, Hkv), 7, dtype=torch.int32, device=DEV)
            ctx_sc = torch.zeros((B, Hkv, nbmax), dtype=torch.float32, device=DEV)
            ctx.seer_gate_select(shape, gate, lens_t, qn, None, budget, ctx_idx, ctx_cnt, max_sel, scores_out=ctx_sc)
            got_idx = torch.full_like(ctx_idx, 9)
            got_cnt = torch.full_like(ctx_cnt, 9)
            # first call: scores go to the caller; second call: they stay in the built-in array
            got_sc = torch.zeros_like(ctx_sc) if call == 0 else None
            binding.seer_gate_select_static(0, shape, gate, lens_t, qn, budget, got_idx, got_cnt, max_sel,
                                            scores_out=got_sc)
            torch.cuda.synchronize()
            # against the oracle: scores, and the selection the oracle makes on the GPU's own scores
            want_sc, _ = oracle.scores(bits(qn), bits(wq), bits(kc), [x - 1 for x in n], [int(L) - 1 for L in lens], THETA)
            sc_for_select = (got_sc if got_sc is not None else ctx_sc).cpu().numpy()
            for i in range(B):
                assert np.abs(sc_for_select[i, :, :n[i] - 1] - want_sc[i, :, :n[i] - 1]).max() <= 1e-3, f"call {call}"
            want_idx, want_cnt = oracle.select(sc_for_select, lens, b, budget, max_sel)
            assert np.array_equal(got_cnt.cpu().numpy(), want_cnt), f"call {call}"
            assert np.array_equal(got_idx.cpu().numpy(), want_idx), f"call {call}"
            # against the context entry point
            assert torch.equal(got_cnt, ctx_cnt) and torch.equal(got_idx, ctx_idx), f"call {call}"
            if got_sc is not None:
                for i in range(B):
                    assert torch.equal(got_sc[i, :, :n[i] - 1], ctx_sc[i, :, :n[i] - 1]), f"call {call}"
    finally:
        ctx.close()


def test_static_entry_point_two_kernel_path_uses_the_built_in_array_twice():
    # 9000 compressed keys per unit: beyond the one-kernel gate, so the gate query, the scores and the
    # tickets go through the built-in array (256 + 256 + 2*128*4 + 2*9000*4 bytes of it)
    b, nbmax = 64, 9000
    lens = np.array([nbmax * b - 3], np.int32)
    _two_calls(B=1, Hq=8, Hkv=2, dg=128, b=b, nbmax=nbmax, lens=lens, max_sel=300, seeds=(501, 502))


def test_static_entry_point_one_kernel_path_twice():
    b, nbmax = 64, 700
    lens = np.array([nbmax * b, 333 * b + 1, 2 * b], np.int32)
    _two_calls(B=3, Hq=10, Hkv=2, dg=128, b=b, nbmax=nbmax, lens=lens, max_sel=64, seeds=(503, 504))


def test_static_entry_point_rejects_what_does_not_fit():
    B, Hq, Hkv, d, dg, b = 8, 40, 8, 128, 128, 64
    nbmax = 16384                                    # two-kernel path; 64 units x 16384 scores x 4 B = 4 MiB > 1 MiB
    qn, wq, kc = _inputs(505, 1, Hq, Hkv, d, dg, 8)  # never read: the call must stop on the host
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, THETA, wq, None, kc, nbmax)
    lens_t = torch.full((B,), 64, dtype=torch.int32, device=DEV)
    idx = torch.zeros((B, Hkv, 4), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    with pytest.raises(binding.SeerError) as e:
        binding.seer_gate_select_static(0, shape, gate, lens_t, qn, 256, idx, cnt, 4)
    assert e.value.status == binding.SEER_ERR_WORKSPACE
    assert str(binding.STATIC_SCRATCH_BYTES) in str(e.value)
