"""The allocation-free decode entry point against the ordinary one.

``ccdc_decode_reduce_static`` serves callers that cannot allocate device memory
where they shuffle (a region where cudaMalloc is forbidden or would stall the
device, or a program whose memory was all handed out at start-up): its scratch
is a fixed array inside the library.  It must give exactly what
``ccdc_decode_reduce`` gives with a caller-supplied workspace, also when the
array still holds another call's data, and must refuse what it cannot serve.
This file is collected last so that a failure here cannot hide another test.
"""
import numpy as np
import pytest

from oracle.ccdc_oracle import Oracle
from paper_1805_01993_b200.inputs import values_numpy

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def ccdc():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_1805_01993_b200 import build, ccdc as mod

    build.build_library()
    mod.lib()
    return mod


def both_ways(ccdc, K, r, N, Q, B, dtype, seed):
    plan = ccdc.Plan(K, r, N, Q, B, dtype)
    plan.tune_decode(plan.decode_threads, 10)           # a split whose partial sums go through scratch memory
    assert 0 < plan.workspace_bytes <= ccdc.lib().ccdc_static_scratch_bytes()
    plan.upload()
    part = plan.alloc_partitions()
    v = values_numpy(N, Q, B, dtype, seed=seed)
    plan.fill_partitions(part, torch.from_numpy(v).cuda())
    coded = plan.alloc(plan.coded_bytes)
    plan.encode_fused(part, coded)
    ref = plan.alloc(plan.out_bytes)
    plan.decode_reduce(part, coded, ref, plan.alloc(plan.workspace_bytes))
    got = torch.zeros_like(ref)
    plan.decode_reduce_static(part, coded, got)         # first call on the device: looks the array up
    torch.cuda.synchronize()
    # same kernels, same order of additions: the bits agree for both dtypes
    assert np.array_equal(got.cpu().numpy().view(np.uint32), ref.cpu().numpy().view(np.uint32))
    # and against the CPU oracle
    o = Oracle(K, r, N, Q, B, dtype)
    o.load_values(v)
    o.shuffle()
    expect = o.reduce()
    have = got.cpu().numpy().reshape(expect.shape)
    if dtype == "int32":
        assert np.array_equal(have, expect)
    else:
        _, a64 = o.direct()
        assert np.all(np.abs(have.astype(np.float64) - expect.astype(np.float64)) <= 1e-5 * a64 + 1e-30)
    # the call itself takes no device memory: free bytes are the same before and after it
    got.zero_()
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    plan.decode_reduce_static(part, coded, got)
    free_called = torch.cuda.mem_get_info()[0]
    torch.cuda.synchronize()
    free_after = torch.cuda.mem_get_info()[0]
    assert free_before == free_called == free_after
    assert np.array_equal(got.cpu().numpy().view(np.uint32), ref.cpu().numpy().view(np.uint32))


def test_two_calls_in_a_row_match_the_allocating_entry_point(ccdc):
    # the second call has another shape and split, and finds the first call's data in the array
    both_ways(ccdc, 10, 3, 480, 10, 1024, "float32", seed=1)
    both_ways(ccdc, 8, 3, 112, 8, 4100, "int32", seed=2)
    both_ways(ccdc, 10, 3, 480, 10, 1024, "float32", seed=3)


def test_refuses_what_it_cannot_serve(ccdc):
    # scratch demand above the built-in array
    big = ccdc.Plan(16, 4, 1820, 16, 147456, "float32")
    big.tune_decode(512, 8)                     # eight partial sums of 9 MB each
    assert big.workspace_bytes > ccdc.lib().ccdc_static_scratch_bytes()
    dummy = torch.zeros(64, dtype=torch.float32, device="cuda")
    before = ccdc.num_kernel_launches()
    with pytest.raises(ccdc.CcdcError) as e:
        big.decode_reduce_static([dummy] * 16, dummy, dummy)
    assert e.value.status == ccdc.ESIZE
    # tables not on the device yet: uploading them would allocate
    fresh = ccdc.Plan(10, 3, 480, 10, 256, "float32")
    fresh.tune_decode(fresh.decode_threads, 10)
    with pytest.raises(ccdc.CcdcError) as e:
        fresh.decode_reduce_static([dummy] * 10, dummy, dummy)
    assert e.value.status == ccdc.ESTATE
    assert ccdc.num_kernel_launches() == before
