"""The allocation-free fitness entry point, for callers that cannot get device
memory when they need a fitness value (a framework's caching allocator already
owns the GPU, a plug-in only receives input/output buffers, or cudaMalloc is
off limits because it stalls the device).  It must return exactly what the
workspace-based entry point returns, call after call, although all calls share
one built-in scratch array that is never cleared.

Collected last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2009_03816_b200 import binding

import gpu_util

pytestmark = pytest.mark.gpu


def _inputs(K, N, ld, seed):
    rng = np.random.default_rng(seed)
    x = np.zeros((K, ld), np.float32)
    x[:, :N] = rng.standard_normal((K, N)).astype(np.float32)
    d = (0.5 + 1.5 * rng.random(N)).astype(np.float32)
    t = rng.standard_normal(N).astype(np.float32)
    return [torch.from_numpy(a).cuda() for a in (x, d, t)]


def _with_workspace(dx, dd, dt, N):
    """The existing route: a context with a caller-allocated workspace."""
    sw = binding.Swarm(dx, torch.zeros_like(dx), dx.clone(), N=N, m_max=0.7, m_min=0.7,
                       c1=1.5, c2=1.5, seed=1, flags=binding.PSOPS_QUADRATIC)
    sw.set_quadratic(dd, dt)
    sw.eval_quadratic()
    out = sw.losses()
    sw.close()
    return out


def test_static_scratch_matches_workspace_route_twice_in_a_row():
    gpu_util.ensure_library()
    stream = torch.cuda.current_stream().cuda_stream
    # second problem is smaller and differently shaped, so stale tile sums of
    # the first call would be picked up if the call relied on a clean array
    for K, N, ld, seed in [(8, 300_001, 300_004, 1), (5, 70_003, 70_004, 2), (8, 300_001, 300_004, 3)]:
        dx, dd, dt = _inputs(K, N, ld, seed)
        want = _with_workspace(dx, dd, dt, N)
        loss = torch.full((K,), -1.0, device="cuda")
        binding.psops_quadratic_fitness_static(dx, ld, K, N, dd, dt, loss, stream)
        got = loss.cpu().numpy()
        # the parity tests hold device-evaluated losses to bit equality
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), (K, N)
        assert np.all(got > 0)


def test_static_scratch_unaligned_rows_and_limit():
    gpu_util.ensure_library()
    K, N = 3, 1001
    dx, dd, dt = _inputs(K, N, 1001, 4)                  # ld % 4 != 0: scalar variant
    want = _with_workspace(dx, dd, dt, N)
    loss = torch.zeros(K, device="cuda")
    binding.psops_quadratic_fitness_static(dx, 1001, K, N, dd, dt, loss)
    assert np.array_equal(loss.cpu().numpy().view(np.uint32), want.view(np.uint32))
    # K * ceil(N / 128) beyond the built-in array: refused, nothing written
    big_n = 128 * (binding.PSOPS_STATIC_SCRATCH_DOUBLES // 2) + 1
    before = loss.clone()
    with pytest.raises(binding.PsopsError) as e:
        binding.psops_quadratic_fitness_static(dx, big_n, 2, big_n, dd, dt, loss)
    assert e.value.code == binding.PSOPS_ELIMIT
    with pytest.raises(binding.PsopsError) as e:
        binding.psops_quadratic_fitness_static(dx, 1001, K, N, None, dt, loss)
    assert e.value.code == binding.PSOPS_EINVAL
    # a host buffer where a device buffer belongs is refused before anything is launched
    pinned = torch.zeros(K).pin_memory()
    with pytest.raises(binding.PsopsError) as e:
        binding.psops_quadratic_fitness_static(dx, 1001, K, N, dd, dt, pinned)
    assert e.value.code == binding.PSOPS_EINVAL
    torch.cuda.synchronize()
    assert torch.equal(loss, before)


def test_static_scratch_exactly_at_its_limit():
    """K * ceil(N / 128) equal to the size of the built-in array: the last slot
    is used, the call is accepted and agrees with the workspace route."""
    gpu_util.ensure_library()
    K, N = 2, 128 * (binding.PSOPS_STATIC_SCRATCH_DOUBLES // 2)
    gen = torch.Generator(device="cuda").manual_seed(7)
    dx = torch.randn((K, N), device="cuda", generator=gen)
    dd = torch.rand(N, device="cuda", generator=gen) * 1.5 + 0.5
    dt = torch.randn(N, device="cuda", generator=gen)
    want = _with_workspace(dx, dd, dt, N)
    loss = torch.full((K,), -1.0, device="cuda")
    binding.psops_quadratic_fitness_static(dx, N, K, N, dd, dt, loss)
    assert np.array_equal(loss.cpu().numpy().view(np.uint32), want.view(np.uint32))
    assert K * ((N + 127) // 128) == binding.PSOPS_STATIC_SCRATCH_DOUBLES
