"""The entry point for callers that cannot allocate device memory (``sop_channel_norms_static``).

Some users of the library may not call cudaMalloc while they work: a server that gave all device
memory to its own arena, a loop that cannot afford the device-wide synchronisation an allocation
implies, a plug-in that receives only tensors.  For them the channel norms are also available with
a scratch array built into the library.  This file checks, through the C-ABI, that the variant
returns exactly what ``sop_channel_norms`` returns -- twice in a row, with different inputs, since
the second call finds the first call's partial sums in the shared scratch -- and that it refuses
problems larger than the built-in scratch.  The file name sorts last on purpose: a run that stops at
the first failure has then already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2605_14929_b200 import inputs as I


@pytest.fixture(scope="module")
def B():
    from paper_2605_14929_b200 import build as libbuild
    libbuild.build()
    from paper_2605_14929_b200 import binding
    binding.lib()
    return binding


def test_too_large_is_refused_on_the_host(B):
    # ceil(T / 64) * K doubles must fit the built-in scratch; the check comes before any CUDA call,
    # so the pointers are never touched
    fake = C.c_void_p(0x10000)
    ll = C.c_longlong
    lib = B.lib()
    K = 14336
    too_many_tokens = 64 * (B.NORMS_STATIC_DOUBLES // K + 1)
    assert lib.sop_channel_norms_static(fake, ll(too_many_tokens), ll(K), ll(K), fake, None) == -8
    assert b"no-allocation" in lib.sop_strerror(-8)
    assert lib.sop_channel_norms_static(None, ll(4), ll(16), ll(16), fake, None) == -1
    assert lib.sop_channel_norms_static(fake, ll(4), ll(16), ll(8), fake, None) == -2


@pytest.mark.gpu
def test_static_scratch_variant_matches_the_workspace_variant_twice(B):
    dev = torch.device("cuda:0")
    # two calls in a row on different inputs and shapes: the second one runs over the first one's leftovers
    for seed, (T, K) in enumerate([(200, 4096), (65, 1040)]):
        X = I.activations(40 + seed, 0, T, K).to(dev)
        want = torch.empty(K, dtype=torch.float32, device=dev)
        ws = B.alloc_workspace(B.channel_norms_workspace(T, K), dev)
        B.sop_channel_norms(X, want, ws)
        got = torch.full((K,), -1.0, dtype=torch.float32, device=dev)
        B.sop_channel_norms_static(X, got)
        torch.cuda.synchronize()
        # same kernels, same order of operations: the tolerance of the other channel-norm tests is bit equality
        assert np.array_equal(got.cpu().numpy().view(np.uint32), want.cpu().numpy().view(np.uint32))
    # the largest problem that fits (ceil(T / 64) * K = 2^19 exactly) is accepted and agrees too
    T, K = 64 * 128, 4096
    X = I.activations(42, 0, T, K).to(dev)
    want = torch.empty(K, dtype=torch.float32, device=dev)
    B.sop_channel_norms(X, want, B.alloc_workspace(B.channel_norms_workspace(T, K), dev))
    got = torch.empty(K, dtype=torch.float32, device=dev)
    B.sop_channel_norms_static(X, got)
    torch.cuda.synchronize()
    assert np.array_equal(got.cpu().numpy().view(np.uint32), want.cpu().numpy().view(np.uint32))
    with pytest.raises(B.SopError) as err:
        B.sop_channel_norms_static(torch.empty((64 * 129, 4096), dtype=torch.float32, device=dev), got)
    assert err.value.code == -8
