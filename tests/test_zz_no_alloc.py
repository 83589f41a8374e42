"""fosgd_decode_noalloc: the decoder for callers that may not allocate device memory (code
living inside someone else's memory pool, loops where cudaMalloc's implicit synchronisation
is banned, processes with no memory left to request).  Its scratch is a fixed array inside the
library, so the test calls it twice in a row, on different inputs, and expects exactly what
fosgd_decode produces with a caller-provided scratch buffer; the second call must not be
disturbed by what the first left in the shared array.  Runs last on purpose."""
import numpy as np
import pytest
import torch

from parity import L2_RTOL

pytestmark = pytest.mark.gpu


def test_noalloc_decoder_matches_decoder_twice():
    import paper_2405_11095_b200 as F

    lib = F.lib()
    stream = torch.cuda.current_stream().cuda_stream
    seed, step, lam = 2024, 9, 0.0625
    # first a transform that needs scratch (2^18 > one tile), then a longer one, then a short one
    for call, (d, wid) in enumerate([((1 << 18) - 5, 3), (1 << 20, 4), (3000, 5)]):
        dp = F.padded_dim(d)
        rng = np.random.default_rng(100 + call)
        words = rng.integers(0, 2 ** 32, dp // 32, dtype=np.uint64).astype(np.uint32)
        bits = torch.from_numpy(words.view(np.int32)).cuda()
        ref = torch.empty(d, dtype=torch.float32, device="cuda")
        ws_bytes = F.workspace_bytes(F.OP_DECODE, d)
        ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")
        F.decode(bits, d, ref, lam, seed, step, wid, ws=ws)
        out = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        # free device memory as the driver reports it (this sees a cudaMalloc made by anyone in the
        # process, which torch's own counters would not); the first call on a device may still load
        # the library's kernels, so the comparison starts with the second
        before = (torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0])
        status = lib.fosgd_decode_noalloc(bits.data_ptr(), d, wid, seed, step, lam, 0, out.data_ptr(), stream)
        assert status == F.OK
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before[0]
        if call > 0:
            assert torch.cuda.mem_get_info()[0] == before[1]
        err = (out.double() - ref.double()).norm() / ref.double().norm()
        assert float(err) <= L2_RTOL
        assert torch.equal(out, ref)      # same kernels, same order: bit identical


def test_noalloc_decoder_rejects_oversize():
    import paper_2405_11095_b200 as F

    d = (1 << 20) + 1                      # pads to 2^21 coordinates: beyond the built-in scratch
    bits = torch.zeros(F.padded_dim(d) // 32, dtype=torch.int32, device="cuda")
    out = torch.zeros(d, dtype=torch.float32, device="cuda")
    with pytest.raises(F.FosgdError) as e:
        F.decode_noalloc(bits, d, out, 0.5, 1, 2, 3)
    assert e.value.status == F.ELIMIT
    assert "2^20" in str(e.value)
    assert not out.any()                   # nothing was enqueued
    # the decoder's own argument checks come before the size limit
    lib = F.lib()
    stream = torch.cuda.current_stream().cuda_stream
    assert lib.fosgd_decode_noalloc(0, d, 3, 1, 2, 0.5, 0, out.data_ptr(), stream) == F.EINVAL
    assert lib.fosgd_decode_noalloc(bits.data_ptr(), d, 3, 1, 2, -1.0, 0, out.data_ptr(), stream) == F.EINVAL
    assert lib.fosgd_decode_noalloc(bits.data_ptr() + 4, d, 3, 1, 2, 0.5, 0, out.data_ptr(), stream) == F.EALIGN
    # blocks of 2^15 are single-pass transforms: no scratch, so no limit on d'
    bits15 = torch.zeros(F.padded_dim(d, 15) // 32, dtype=torch.int32, device="cuda")
    ref = torch.empty(d, dtype=torch.float32, device="cuda")
    F.decode(bits15, d, ref, 0.5, 1, 2, 3, block_log2=15)
    F.decode_noalloc(bits15, d, out, 0.5, 1, 2, 3, block_log2=15)
    torch.cuda.synchronize()
    assert torch.equal(out, ref)
