"""The linear entry point that allocates nothing (needs a B200).

Some users of this library run where device allocation is not allowed at call time: a serving
loop whose memory pool is fixed once at start-up, a plug-in that owns only the buffers it was
handed, code between the begin and end of a latency-critical section. spec_op_linear needs a
scratch buffer from its caller; spec_op_linear_static keeps that scratch inside the library.
This file checks, through the C ABI, that the second gives the first's result, twice in a row
(the built-in scratch still holds the first call's partial sums when the second call starts),
and that a problem larger than the built-in scratch is refused with a message.

Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = 1e-5   # the tolerance of the stand-alone linear tests: max|a-b| / max|b|


@pytest.fixture(scope="module")
def torch():
    t = pytest.importorskip("torch")
    if not t.cuda.is_available():
        pytest.skip("no CUDA device")
    return t


def _operands(torch, M, N, K, seed, dtype):
    rng = np.random.default_rng(seed)
    x = torch.from_numpy(rng.standard_normal((M, K)).astype(np.float32)).cuda().to(dtype)
    w = torch.from_numpy((rng.standard_normal((N, K)) * 0.05).astype(np.float32)).cuda().to(dtype)
    return x, w


def test_static_scratch_linear_matches_caller_scratch_linear_twice(torch):
    from paper_2503_14153_b200 import spec_op_linear, spec_op_linear_static
    # two different problems back to back: the second starts with the first's leftovers in the scratch
    cases = [(64, 1000, 704, 3, 11), (32, 384, 256, 2, 12)]
    for M, N, K, ctas, seed in cases:
        x, w = _operands(torch, M, N, K, seed, torch.bfloat16)
        want = spec_op_linear(x, w, ctas)
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")   # caller-owned output
        before = torch.cuda.memory_stats()["allocation.all.allocated"]    # cumulative count of allocations
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]                        # what the driver says is free on the device
        got = spec_op_linear_static(x, w, y, ctas)
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == before   # none came from torch's allocator
        if (M, N, K) != cases[0][:3]:
            # (the library links the CUDA runtime statically, so an allocation of its own would not show in torch's
            # counters: after the first call, which may load the kernels' code, the device's free memory must not move)
            assert torch.cuda.mem_get_info()[0] == free_before
        torch.cuda.synchronize()
        err = (got - want).abs().max().item() / want.abs().max().item()
        assert err <= TOL, (M, N, K, ctas, err)
    # the same problem again: identical bits both times
    x, w = _operands(torch, 64, 1000, 704, 11, torch.bfloat16)
    y1 = spec_op_linear_static(x, w, torch.empty((64, 1000), dtype=torch.float32, device="cuda"), 3).clone()
    y2 = spec_op_linear_static(x, w, torch.empty((64, 1000), dtype=torch.float32, device="cuda"), 3)
    assert torch.equal(y1, y2)


def test_static_scratch_linear_float32(torch):
    from paper_2503_14153_b200 import spec_op_linear, spec_op_linear_static
    x, w = _operands(torch, 13, 301, 688, 13, torch.float32)
    want = spec_op_linear(x, w)
    got = spec_op_linear_static(x, w, torch.empty((13, 301), dtype=torch.float32, device="cuda"))
    assert (got - want).abs().max().item() / want.abs().max().item() <= TOL


def test_static_scratch_linear_refuses_oversize(torch):
    from paper_2503_14153_b200 import SpecError, spec_op_linear_static
    from paper_2503_14153_b200.binding import STATIC_SCRATCH_FLOATS
    M, N, K, ctas = 64, 32768, 256, 4
    from paper_2503_14153_b200 import load_library
    assert load_library().spec_op_linear_scratch_floats(M, N, K, ctas) > STATIC_SCRATCH_FLOATS
    x, w = _operands(torch, M, N, K, 14, torch.bfloat16)
    y = torch.empty((M, N), dtype=torch.float32, device="cuda")
    with pytest.raises(SpecError) as ei:
        spec_op_linear_static(x, w, y, ctas)
    assert ei.value.code == -3 and "exceeds the built-in scratch" in str(ei.value)
