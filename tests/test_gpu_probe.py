"""The read-bandwidth diagnostic reads every byte it is given exactly once: its checksum is the
exclusive-or of the buffer's 32-bit words (numpy on a host copy of the same bits)."""
import numpy as np
import pytest
import torch

from paper_2506_08889_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("n_words", [0, 4, 4 * 37, 4 * (512 * 8 * 3 + 5), 4 * 1_300_003])
def test_checksum_covers_every_word_once(n_words):
    ctx = binding.Context(0)
    try:
        r = synth.np_rng(5, f"probe{n_words}")
        host = r.integers(0, 2 ** 32, size=max(n_words, 4), dtype=np.uint32)
        buf = torch.from_numpy(host.view(np.int32).copy()).to(DEV)
        chk = torch.full((1,), -1, dtype=torch.int64, device=DEV)
        ctx.seer_debug_read_bandwidth(buf, 4 * n_words, chk)
        torch.cuda.synchronize()
        want = int(np.bitwise_xor.reduce(host[:n_words])) if n_words else 0
        assert int(chk.item()) == want
        with pytest.raises(binding.SeerError):
            ctx.seer_debug_read_bandwidth(buf, 4 * n_words + 8, chk)          # not a multiple of 16 bytes
    finally:
        ctx.close()
