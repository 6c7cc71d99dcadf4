"""The allocation-free entry point against the context-based one.

dipaco_module_sync_static serves callers that cannot use the device allocator (all device memory
already handed to their own pool, or a loop that cannot take cudaMalloc's device-wide
synchronisation): its partial sums live in a static device array inside the library.  It must
give the same module update as dipaco_outer_sync on a one-level, one-module grid, on two calls in
a row (the static array is reused and keeps the first call's contents).

This file sorts last on purpose, so a run that stops at the first failure has already run every
other test.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

from paper_2403_10616_b200 import binding as B
from tests import helpers

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def reference_sync(theta, momentum, copies, weights, reported, dtype, chunk):
    code = B.DIPACO_BF16 if dtype == torch.bfloat16 else B.DIPACO_F32
    P = len(copies)
    ctx = B.dipaco_create((1,), (theta.numel(),), np.zeros((P, 1), np.int32), weights,
                          np.float32(0.7), np.float32(0.9), code, chunk, 0)
    B.dipaco_outer_sync(ctx, theta.data_ptr(), momentum.data_ptr(), [c.data_ptr() for c in copies],
                        reported)
    assert B.dipaco_device_status(ctx) == B.DIPACO_OK
    B.dipaco_destroy(ctx)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_static_scratch_entry_point_matches_the_context_based_one_twice(dtype):
    numel, P, chunk = 50_003, 20, 8
    gen = torch.Generator(device=DEV)
    gen.manual_seed(7)
    theta = torch.empty(numel, device=DEV).normal_(0, 0.02, generator=gen)
    momentum = torch.empty(numel, device=DEV).normal_(0, 1e-4, generator=gen)
    rng = np.random.RandomState(1)
    weights = rng.randint(1000, 10001, size=P).astype(np.float32)
    reported = np.ones(P, dtype=np.uint8)
    reported[[3, 17]] = 0
    code = B.DIPACO_BF16 if dtype == torch.bfloat16 else B.DIPACO_F32

    ref = (theta.clone(), momentum.clone())
    got = (theta.clone(), momentum.clone())
    for call in range(2):
        # a fresh inner phase: every copy drifts away from the current module value
        drift = [torch.empty(numel, device=DEV).normal_(0, 1e-3, generator=gen) for _ in range(P)]
        ref_copies = [(ref[0] + d).to(dtype) for d in drift]
        got_copies = [c.clone() for c in ref_copies]
        reference_sync(ref[0], ref[1], ref_copies, weights, reported, dtype, chunk)
        B.dipaco_module_sync_static(got[0].data_ptr(), got[1].data_ptr(), numel,
                                    [c.data_ptr() for c in got_copies], weights, reported,
                                    np.float32(0.7), np.float32(0.9), code, chunk, 0)
        torch.cuda.synchronize()
        for a, b in ((got[0], ref[0]), (got[1], ref[1])):
            err = (a.double() - b.double()).abs()
            assert bool((err <= 1e-6 * (1 + b.double().abs())).all())
            assert torch.equal(a.view(torch.int32), b.view(torch.int32))
        bits = torch.int16 if dtype == torch.bfloat16 else torch.int32
        for a, b in zip(got_copies, ref_copies):
            assert torch.equal(a.view(bits), b.view(bits))
        assert not torch.equal(got[0], theta)


def test_static_scratch_entry_point_with_nobody_reporting_and_limits():
    numel, P = 4097, 5
    theta = torch.randn(numel, device=DEV) * 0.02
    momentum = torch.randn(numel, device=DEV) * 1e-4
    copies = [torch.zeros(numel, device=DEV) for _ in range(P)]
    t0, m0 = theta.clone(), momentum.clone()
    B.dipaco_module_sync_static(theta.data_ptr(), momentum.data_ptr(), numel,
                                [c.data_ptr() for c in copies], None, np.zeros(P, np.uint8),
                                0.7, 0.9, B.DIPACO_F32, 2, 0)
    torch.cuda.synchronize()
    assert torch.equal(theta, t0) and torch.equal(momentum, m0)
    for c in copies:
        assert torch.equal(c, t0)
    # beyond the static array: refused before anything is launched
    with pytest.raises(B.DipacoError) as e:
        B.dipaco_module_sync_static(theta.data_ptr(), momentum.data_ptr(),
                                    B.DIPACO_STATIC_MAX_NUMEL + 1, [c.data_ptr() for c in copies])
    assert e.value.status == B.DIPACO_ELIMIT
    assert "limit" in str(e.value)
    with pytest.raises(B.DipacoError) as e:
        B.dipaco_module_sync_static(theta.data_ptr(), momentum.data_ptr(), numel,
                                    [c.data_ptr() for c in copies], chunk_paths=33)
    assert e.value.status == B.DIPACO_EINVAL
    torch.cuda.synchronize()
    assert torch.equal(theta, t0)


CASES = {
    # name: (num_paths, chunk_paths, paths that did not report, all weights zero, side stream)
    "first_chunk_silent": (20, 8, list(range(0, 8)), False, False),
    "middle_chunk_silent": (20, 8, list(range(8, 16)), False, False),
    "one_chunk_reports": (20, 8, list(range(0, 8)) + list(range(16, 20)), False, False),
    "single_chunk": (6, 8, [4], False, False),
    "zero_total_weight": (12, 5, [], True, False),
    "side_stream": (20, 8, [3, 17], False, True),
}


@pytest.mark.parametrize("case", sorted(CASES))
def test_static_scratch_entry_point_masks_weights_streams_oracle_and_no_allocation(case):
    """Masks that silence whole chunks, a single chunk, zero total weight and a caller's stream:
    each bitwise equal to the context-based call and within the fp32 tolerance of the oracle; and
    the call itself takes no device memory (free memory is the same before and after a call, once
    the set-up call has loaded the module)."""
    P, chunk, silent, zero_weights, side = CASES[case]
    numel = 12_345
    gen = torch.Generator(device=DEV)
    gen.manual_seed(11)
    theta = torch.empty(numel, device=DEV).normal_(0, 0.02, generator=gen)
    momentum = torch.empty(numel, device=DEV).normal_(0, 1e-4, generator=gen)
    copies = [(theta + torch.empty(numel, device=DEV).normal_(0, 1e-3, generator=gen)).to(torch.bfloat16)
              for _ in range(P)]
    rng = np.random.RandomState(2)
    weights = np.zeros(P, np.float32) if zero_weights else rng.randint(1, 100, size=P).astype(np.float32)
    reported = np.ones(P, dtype=np.uint8)
    reported[silent] = 0

    th0 = helpers.tensor_to_numpy(theta)
    mo0 = helpers.tensor_to_numpy(momentum)
    ps0 = [helpers.tensor_to_numpy(c) for c in copies]

    ref = (theta.clone(), momentum.clone(), [c.clone() for c in copies])
    reference_sync(ref[0], ref[1], ref[2], weights, reported, torch.bfloat16, chunk)

    stream = torch.cuda.Stream() if side else None
    # set-up call on scratch data (loads the module, looks the array up), then the measured call
    warm = (theta.clone(), momentum.clone(), [c.clone() for c in copies])
    B.dipaco_module_sync_static(warm[0].data_ptr(), warm[1].data_ptr(), numel,
                                [c.data_ptr() for c in warm[2]], weights, reported,
                                np.float32(0.7), np.float32(0.9), B.DIPACO_BF16, chunk, 0)
    got = (theta.clone(), momentum.clone(), [c.clone() for c in copies])
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    if side:
        stream.wait_stream(torch.cuda.current_stream())
    B.dipaco_module_sync_static(got[0].data_ptr(), got[1].data_ptr(), numel,
                                [c.data_ptr() for c in got[2]], weights, reported,
                                np.float32(0.7), np.float32(0.9), B.DIPACO_BF16, chunk, 0,
                                stream=stream)
    if side:
        stream.synchronize()
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before

    assert torch.equal(got[0].view(torch.int32), ref[0].view(torch.int32))
    assert torch.equal(got[1].view(torch.int32), ref[1].view(torch.int32))
    for a, b in zip(got[2], ref[2]):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))

    import oracle
    want_th, want_mo, want_ps = th0.copy(), mo0.copy(), [p.copy() for p in ps0]
    oracle.outer_sync((1,), (numel,), np.zeros((P, 1), np.int32), want_th, want_mo, want_ps,
                      oracle.BF16, float(np.float32(0.7)), float(np.float32(0.9)), weights, reported, 4)
    for a, want in ((got[0], want_th), (got[1], want_mo)):
        g = helpers.tensor_to_numpy(a).astype(np.float64)
        assert np.all(np.abs(g - want) <= 1e-6 * (1.0 + np.abs(want.astype(np.float64))))
    for a, want in zip(got[2], want_ps):
        helpers.assert_bf16_copies_close(helpers.tensor_to_numpy(a), want)
    if zero_weights:
        assert torch.equal(got[0], theta) and torch.equal(got[1], momentum)
