"""a2cid2_consensus_distance_static, the entry point for callers that may not allocate.

Some programs cannot let a library call cudaMalloc once they are running: their own memory pool
already owns the device, or they sit in a loop that cannot afford the device-wide stall an
allocation may cause. For them the library offers the consensus distance with its scratch in a
fixed array inside the library instead of in allocated memory. This test calls it through the C
ABI twice in a row, on different data and sizes, and compares each result with the handle-based
a2cid2_consensus_distance on the same rows and with the CPU checker's reduction of the same rows
(a fault shared by the two device entry points would pass the first comparison alone), within the
tolerance the other consensus tests use. The second call uses fewer partial sums than the first, so
anything the first call left in the shared array would show up as a wrong sum; and the free device
memory is read before and after that second call, since the point of the entry point is that it
takes none.

The file is named so that pytest collects it last; it needs nothing from the other tests and
passes on its own in a fresh process as well as after them.
"""
import numpy as np
import pytest

from oracle.sim import OracleSim
from paper_2306_08289_b200 import binding as B
from paper_2306_08289_b200 import workload as W

pytestmark = pytest.mark.gpu

REL_TOL = 2e-6  # as in the consensus-distance parity tests


def _reference(n, d, storage, rows):
    """The existing entry point on the same rows (engine buffers allocated through torch)."""
    eng = B.Engine(n, d, 0.1, 0.5, 0.5, 0.0, storage=storage, n_grad_slots=0)
    eng.write_state(rows)
    return eng, eng.consensus_distance()


@pytest.mark.parametrize("storage", ["f32", "bf16"])
def test_static_scratch_matches_allocating_entry_point_twice(storage):
    import torch

    rng = np.random.default_rng(2024)
    out = torch.zeros(2, dtype=torch.float64, device="cuda:0")  # the caller's output buffer
    stream = torch.cuda.current_stream().cuda_stream
    code = B.A2_BF16 if storage == "bf16" else B.A2_F32
    results = []
    for k, (n, d) in enumerate([(12, 300_007), (5, 4_099)]):  # many partials, then few
        rows = (rng.standard_normal((n, d)) * (k + 1.0) + 0.5).astype(np.float32)
        if storage == "bf16":
            rows = W.f32_to_bf16_bits(rows)
        eng, want = _reference(n, d, storage, rows)
        wide = W.bf16_bits_to_f32(rows).astype(np.float64) if storage == "bf16" else rows.astype(np.float64)
        checker = OracleSim(wide, 0.0, 0.5, 0.5, 0.0).consensus()
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        B.consensus_distance_static(eng.x.data_ptr(), n, d, eng.pitch, code, stream, out[k:].data_ptr())
        torch.cuda.synchronize()
        free_after = torch.cuda.mem_get_info()[0]
        if k == 1:  # the first call on a device may load the kernels; later calls take nothing
            assert free_after == free_before, (free_before, free_after)
        got = float(out[k].item())
        results.append((got, want, checker))
        eng.close()
    for got, want, checker in results:
        assert want > 0 and abs(got - want) <= REL_TOL * want, (got, want)
        assert abs(got - checker) <= REL_TOL * checker, (got, checker)


def test_static_scratch_rejects_what_it_cannot_hold():
    import torch

    buf = torch.zeros(64, dtype=torch.float32, device="cuda:0")
    out = torch.zeros(1, dtype=torch.float64, device="cuda:0")
    s = torch.cuda.current_stream().cuda_stream
    # a width beyond the fixed array's reach is refused on the host: nothing is launched, so the
    # (far too small) buffer is never touched
    with pytest.raises(B.A2Error) as e:
        B.consensus_distance_static(buf.data_ptr(), 2, 67_108_865, 67_108_872, B.A2_F32, s, out.data_ptr())
    assert e.value.code == B.A2_ERANGE and "exceeds" in str(e.value)
    for args in [(None, 2, 8, 8, B.A2_F32, s, out.data_ptr()),            # no input
                 (buf.data_ptr(), 1, 8, 8, B.A2_F32, s, out.data_ptr()),  # one worker
                 (buf.data_ptr(), 2, 9, 8, B.A2_F32, s, out.data_ptr()),  # pitch < d
                 (buf.data_ptr(), 2, 8, 12, B.A2_F32, s, out.data_ptr()),  # pitch not a multiple of 8
                 (buf.data_ptr() + 4, 2, 8, 8, B.A2_F32, s, out.data_ptr()),  # misaligned
                 (buf.data_ptr(), 2, 8, 8, 9, s, out.data_ptr()),         # unknown storage type
                 (buf.data_ptr(), 2, 8, 8, B.A2_F32, s, None)]:           # no output
        with pytest.raises(B.A2Error) as e:
            B.consensus_distance_static(*args)
        assert e.value.code == B.A2_EINVAL
    torch.cuda.synchronize()
    assert float(out.item()) == 0.0
