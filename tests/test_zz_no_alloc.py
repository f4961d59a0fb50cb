"""rtma_partition_static: the partition for callers that cannot allocate device memory.

Some users of the library partition at a moment when cudaMalloc is off limits (a fixed memory
budget pinned at start-up, a lock under which nothing may synchronise the device, a stream that
is about to be captured).  For them the library offers a variant whose scratch is a fixed array
inside the library.  This file checks, through the C ABI, that the variant gives exactly the
result of rtma_partition, twice in a row (the second call meets the first call's leftovers in the
shared scratch), and that it refuses sizes beyond its fixed scratch.  It is collected last so a
failure here cannot hide the result of any other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2305_09887_b200 import binding

pytestmark = pytest.mark.gpu


def _same(a, b):
    return all(torch.equal(x, y) for x, y in zip(a, b))


def test_static_partition_matches_partition_twice_in_a_row():
    ctx = binding.Context(0)
    # first call: close to the scratch limit (4096 chunks x 64 parts), node-level assignment
    n1, M1, seed1 = 4_000_000, 64, 0x5EED0005
    got1 = binding.partition_static(n1, None, seed1, M1)
    torch.cuda.synchronize()
    want1 = ctx.partition(n1, None, seed1, M1)
    torch.cuda.synchronize()
    assert _same(got1, want1)
    # second call straight after, smaller and with super-node ids: stale scratch must not matter
    n2, M2, seed2 = 300_001, 7, 99
    group = torch.from_numpy((np.random.default_rng(1).integers(0, 3000, size=n2) * 5 - 11).astype(np.int32)).cuda()
    got2 = binding.partition_static(n2, group, seed2, M2)
    torch.cuda.synchronize()
    want2 = ctx.partition(n2, group, seed2, M2)
    torch.cuda.synchronize()
    assert _same(got2, want2)
    # and the first problem again gives the first answer again
    got3 = binding.partition_static(n1, None, seed1, M1)
    torch.cuda.synchronize()
    assert _same(got3, want1)
    # empty input
    e = binding.partition_static(0, None, 1, 4)
    torch.cuda.synchronize()
    assert e[1].cpu().tolist() == [0] * 5


def test_static_partition_at_the_limit_allocates_nothing():
    # exactly ceil(n / 1024) * M = the fixed scratch's cell count, outputs provided by the caller: the
    # call works, agrees with rtma_partition bit for bit, and leaves the device's free memory as it was
    lib = binding.load_library()
    n, M, seed = 4096 * 1024, 64, 17
    assert ((n + 1023) // 1024) * M == binding.PARTITION_STATIC_MAX_CELLS
    dev = torch.device("cuda", 0)
    out = [torch.empty(n, dtype=torch.int32, device=dev), torch.empty(M + 1, dtype=torch.int64, device=dev),
           torch.empty(n, dtype=torch.int32, device=dev), torch.empty(n, dtype=torch.int32, device=dev)]

    def call():
        st = lib.rtma_partition_static(ctypes.c_int32(0), ctypes.c_int64(n), ctypes.c_void_p(0), ctypes.c_uint64(seed),
                                       ctypes.c_int32(M), *[ctypes.c_void_p(t.data_ptr()) for t in out],
                                       ctypes.c_void_p(int(torch.cuda.current_stream().cuda_stream)))
        assert st == 0, lib.rtma_partition_static_error()
        torch.cuda.synchronize()

    call()                                  # the first call on a device looks the scratch's address up
    free_before, _ = torch.cuda.mem_get_info(dev)
    call()
    free_after, _ = torch.cuda.mem_get_info(dev)
    assert free_after == free_before        # no device memory taken or returned by the call
    ctx = binding.Context(0)
    want = ctx.partition(n, None, seed, M)
    torch.cuda.synchronize()
    assert _same(out, want)


def test_static_partition_rejects_sizes_beyond_its_scratch():
    lib = binding.load_library()
    n, M = 1024 * 4097, 64      # 4097 chunks x 64 parts > 262144 cells
    assert ((n + 1023) // 1024) * M > binding.PARTITION_STATIC_MAX_CELLS
    dummy = torch.zeros(8, dtype=torch.int64, device="cuda")
    p = ctypes.c_void_p(dummy.data_ptr())
    st = lib.rtma_partition_static(ctypes.c_int32(0), ctypes.c_int64(n), ctypes.c_void_p(0), ctypes.c_uint64(1),
                                   ctypes.c_int32(M), p, p, p, p, ctypes.c_void_p(0))
    assert st == -3                                          # RTMA_ERR_WORKSPACE, nothing launched
    assert b"exceeds the fixed scratch" in lib.rtma_partition_static_error()
    torch.cuda.synchronize()
    assert dummy.abs().sum().item() == 0
    with pytest.raises(binding.RtmaError):
        binding.partition_static(n, None, 1, M)
