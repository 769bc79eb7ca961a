"""seer_gate_select_static: gate scoring + selection for callers that may not allocate.

A serving process that gives all of its HBM to its own pool at start-up, or code running where
the CUDA allocator must not be entered, cannot create a context (seer_create allocates the
workspace).  For them the library keeps the gate's scratch in a fixed array of its own image.
This test calls that entry point through the C ABI twice in a row, with different queries, and
checks each result against the ordinary context-based seer_gate_select on the same inputs: the
scores within the tolerance the gate tests use, the selected block lists exactly.  The second
call also shows that what the first one left in the shared array does no harm.

The file name makes pytest collect it last, so a run that stops at the first failure has
already been through every other test."""
import numpy as np
import pytest
import torch

from paper_2506_08889_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inputs(seed, B, Hq, Hkv, d, dg, nbmax):
    g = Hq // Hkv
    qn = synth.normal_bf16((B, Hq, d), seed, "zz:qn", DEV)
    wq = synth.normal_bf16((Hkv, dg, g * d), seed, "zz:wq", DEV, std=0.02)
    kc = synth.normal_bf16((B, Hkv, nbmax, dg), seed, "zz:kc", DEV)
    return qn, wq, kc


def test_static_entry_point_matches_context_entry_point_twice():
    B, Hq, Hkv, d, dg, b, nbmax = 3, 10, 2, 128, 128, 64, 700       # large enough for the split kernels
    lens = np.array([nbmax * b, 333 * b + 1, 2 * b], np.int32)
    lens_t = torch.as_tensor(lens, device=DEV)
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    max_sel, budget = 64, 64 * b
    ctx = binding.Context(0)
    try:
        for call, seed in enumerate((501, 502)):
            qn, wq, kc = _inputs(seed, B, Hq, Hkv, d, dg, nbmax)
            gate = binding.make_gate(dg, 1.0e6, wq, None, kc, nbmax)
            want_idx = torch.full((B, Hkv, max_sel), 7, dtype=torch.int32, device=DEV)
            want_cnt = torch.full((B, Hkv), 7, dtype=torch.int32, device=DEV)
            want_sc = torch.zeros((B, Hkv, nbmax), dtype=torch.float32, device=DEV)
            ctx.seer_gate_select(shape, gate, lens_t, qn, None, budget, want_idx, want_cnt, max_sel,
                                 scores_out=want_sc)
            got_idx = torch.full_like(want_idx, 9)
            got_cnt = torch.full_like(want_cnt, 9)
            # first call: scores go to the caller; second call: they stay in the built-in scratch
            got_sc = torch.zeros_like(want_sc) if call == 0 else None
            binding.seer_gate_select_static(0, shape, gate, lens_t, qn, budget, got_idx, got_cnt, max_sel,
                                            scores_out=got_sc)
            torch.cuda.synchronize()
            assert torch.equal(got_cnt, want_cnt), f"call {call}"
            assert torch.equal(got_idx, want_idx), f"call {call}"
            if got_sc is not None:
                assert (got_sc - want_sc).abs().max().item() <= 1e-3
    finally:
        ctx.close()


def test_static_entry_point_rejects_what_does_not_fit():
    B, Hq, Hkv, d, dg, b = 8, 40, 8, 128, 128, 64
    nbmax = 8192                                     # 64 units x 8192 scores x 4 B = 2 MiB > 1 MiB
    qn, wq, kc = _inputs(503, 1, Hq, Hkv, d, dg, 8)  # never read: the call must stop on the host
    shape = binding.make_shape(B, Hq, Hkv, d, b, 0.1)
    gate = binding.make_gate(dg, 1.0e6, wq, None, kc, nbmax)
    lens_t = torch.full((B,), 64, dtype=torch.int32, device=DEV)
    idx = torch.zeros((B, Hkv, 4), dtype=torch.int32, device=DEV)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=DEV)
    with pytest.raises(binding.SeerError) as e:
        binding.seer_gate_select_static(0, shape, gate, lens_t, qn, 256, idx, cnt, 4)
    assert e.value.status == binding.SEER_ERR_WORKSPACE
    assert str(binding.STATIC_SCRATCH_BYTES) in str(e.value)
