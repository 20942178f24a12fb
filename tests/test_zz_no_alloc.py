"""ah_distances_static: the entry point for callers that must not allocate device memory
(a hook inside a job whose framework already owns the whole GPU, a latency-critical loop,
a component that has raw pointers but no handle).  It keeps its per-tile partial sums in
a fixed array inside the library instead of a workspace.

The check: called through the C ABI, twice in a row (the array is shared between calls
and keeps the first call's contents), it must return exactly what the handle-based path
returns for the same x and c, bit for bit, which is the tolerance the other distance
tests use.  This file is collected last, so a run that stops at the first failure has
already been through every other test."""
import numpy as np
import pytest

from paper_2409_09242_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _handle_distances(B, torch, x, c):
    """||x_i - c||^2 through the existing entry points: load x and c into a handle and
    take a step in which no worker is active but distances are wanted."""
    K, P = x.shape
    h = B.Handle(K, P, [])
    h.ah_state_set(B.AH_CENTER, c)
    h.ah_state_set(B.AH_X, x)
    z = torch.zeros((K, W.padded_ld(P)), device="cuda")
    h.ah_local_step(z, z, 1, lr=0.0, active=np.zeros(K, np.uint8), want_dist=True)
    out = h.ah_state_get(B.AH_NORM2).copy()
    h.close()
    return out


def test_static_scratch_distances_match_handle_path_twice():
    import torch
    from paper_2409_09242_b200 import binding as B
    torch.cuda.set_device(0)
    rng = np.random.default_rng(2024)
    out = torch.empty(8, dtype=torch.float64, device="cuda")
    # two different problems back to back: the second must not see the first's partials
    for K, P in ((4, 300_001), (8, 5_000), (3, 1), (2, 1 << 20)):
        ld = W.padded_ld(P)
        c = rng.standard_normal(P).astype(np.float32)
        x = c[None] + rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.02)
        want = _handle_distances(B, torch, x, c)
        xd = torch.zeros((K, ld), device="cuda")
        xd[:, :P] = torch.from_numpy(x)
        cd = torch.zeros(ld, device="cuda")
        cd[:P] = torch.from_numpy(c)
        for call in range(2):
            out.fill_(-1.0)
            B.ah_distances_static(xd[:, :P], cd, out)
            torch.cuda.synchronize()
            got = out[:K].cpu().numpy()
            assert np.array_equal(got, want), (K, P, call)
            assert np.all(got > 0)


def test_static_scratch_rejects_what_does_not_fit():
    import torch
    from paper_2409_09242_b200 import binding as B
    torch.cuda.set_device(0)
    lib = B.raw()
    buf = torch.zeros(4096, device="cuda")
    out = torch.zeros(256, dtype=torch.float64, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    # capacity: K * pow2(ceil(P / 1024)) <= AH_STATIC_SCRATCH_ENTRIES; pointers are not
    # touched when the size check fails, so a small buffer is enough here
    big_p = 1024 * (B.AH_STATIC_SCRATCH_ENTRIES // 4) + 4
    assert lib.ah_distances_static(buf.data_ptr(), big_p, buf.data_ptr(), 4, big_p, out.data_ptr(),
                                   stream) == B.AH_ERR_TOO_LARGE
    assert "capacity" in B.ah_status_string(B.AH_ERR_TOO_LARGE)
    assert lib.ah_distances_static(buf.data_ptr(), 1024, buf.data_ptr(), 257, 1024, out.data_ptr(),
                                   stream) == B.AH_ERR_INVALID_ARG
    assert lib.ah_distances_static(buf.data_ptr() + 4, 1024, buf.data_ptr(), 2, 1024, out.data_ptr(),
                                   stream) == B.AH_ERR_ALIGN
    assert lib.ah_distances_static(buf.data_ptr(), 1022, buf.data_ptr(), 2, 1022, out.data_ptr(),
                                   stream) == B.AH_ERR_ALIGN
    assert lib.ah_distances_static(None, 1024, buf.data_ptr(), 2, 1024, out.data_ptr(),
                                   stream) == B.AH_ERR_INVALID_ARG
    # a small call still runs after the refusals (x == c: every distance is zero)
    assert lib.ah_distances_static(buf.data_ptr(), 1024, buf.data_ptr(), 4, 1024, out.data_ptr(),
                                   stream) == B.AH_OK
    torch.cuda.synchronize()
    assert np.all(out[:4].cpu().numpy() == 0.0)


def test_static_scratch_at_exactly_its_capacity_and_one_entry_above():
    """K = 128 workers of 2^20 parameters need 128 x 1024 tile sums: every entry of the
    built-in array.  The result must still equal the handle path bit for bit, twice in a
    row; one worker more, or one tile more per worker, is refused."""
    import torch
    from paper_2409_09242_b200 import binding as B
    torch.cuda.set_device(0)
    K, P = 128, 1 << 20
    assert K * (P // 1024) == B.AH_STATIC_SCRATCH_ENTRIES
    gen = torch.Generator(device="cuda").manual_seed(11)
    cd = torch.empty(P, device="cuda").normal_(generator=gen)
    xd = cd[None, :] + torch.empty((K, P), device="cuda").normal_(generator=gen) * 0.02
    # the handle path on the same device arrays
    h = B.Handle(K, P, [])
    h.ah_state_set(B.AH_CENTER, cd)
    h.ah_state_set(B.AH_X, xd)
    z = torch.zeros((K, P), device="cuda")                       # never read: nobody steps
    h.ah_local_step(z, z, 1, lr=0.0, active=np.zeros(K, np.uint8), want_dist=True)
    want = h.ah_state_get(B.AH_NORM2).copy()
    h.close()
    out = torch.empty(K + 1, dtype=torch.float64, device="cuda")
    for call in range(2):
        out.fill_(-1.0)
        B.ah_distances_static(xd, cd, out)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        assert np.array_equal(got[:K], want), call
        assert got[K] == -1.0                                     # nothing written past K
    assert np.all(want > 0) and np.allclose(want, P * 0.02 ** 2, rtol=0.05)
    lib = B.raw()
    stream = torch.cuda.current_stream().cuda_stream
    # one tile more per worker rounds up to 2048 tiles; one worker more needs 129 x 1024
    assert lib.ah_distances_static(xd.data_ptr(), P + 4, cd.data_ptr(), K, P + 4, out.data_ptr(),
                                   stream) == B.AH_ERR_TOO_LARGE
    assert lib.ah_distances_static(xd.data_ptr(), P, cd.data_ptr(), K + 1, P, out.data_ptr(),
                                   stream) == B.AH_ERR_TOO_LARGE
