"""The allocation-free host-gradient local step (collected last on purpose).

Some callers cannot allocate device memory -- for instance code running under a framework whose
caching allocator has already taken the whole GPU, or a latency-critical loop that cannot afford
the device-wide synchronisation an allocation may cause.  For them the library offers one entry
point that stages host gradients through a fixed array inside the library image instead of a
cudaMalloc'ed buffer.  This test calls it through the C boundary and checks, on two calls in a
row, that it produces exactly what the existing entry point (cocod_kernel_local_step, fed the same
gradients from device memory) produces -- the second call also shows that bytes left in the shared
staging array by the first one do no harm."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def E():
    from paper_1906_12043_b200 import build, engine
    build.build()
    engine.load()
    return engine


def test_noalloc_entry_point_matches_the_existing_one_twice_in_a_row(E):
    rng = np.random.default_rng(123)
    lr, mu, wd = 0.1, 0.9, 5e-4
    for call, n in enumerate([1_000_003, 300_001]):       # second call: smaller, staging holds stale bytes
        x = torch.from_numpy((rng.standard_normal(n) * 0.01).astype(np.float32)).cuda()
        v = torch.from_numpy((rng.standard_normal(n) * 0.02).astype(np.float32)).cuda()
        g_host = torch.from_numpy((rng.standard_normal(n) * 0.01).astype(np.float32)).pin_memory()
        # existing entry point, gradients already on the device
        x_ref, v_ref = x.clone(), v.clone()
        E.kernel_local_step(x_ref, x_ref, v_ref, g_host.cuda(), lr, mu, wd)
        # new entry point, gradients in host memory, in place
        x_new, v_new = x.clone(), v.clone()
        E.kernel_local_step_host_noalloc(x_new, x_new, v_new, g_host, lr, mu, wd)
        torch.cuda.synchronize()
        assert torch.equal(x_new.view(torch.int32), x_ref.view(torch.int32)), f"call {call}: x differs"
        assert torch.equal(v_new.view(torch.int32), v_ref.view(torch.int32)), f"call {call}: v differs"
        assert not torch.equal(x_new, x)                   # and it did something


def test_noalloc_entry_point_rejects_oversized_requests_and_bad_arguments(E):
    lib = E.load()
    n = E.NOALLOC_MAX_ELEMS + 1
    dummy = torch.zeros(8, device="cuda")
    host = torch.zeros(8)
    rc = lib.cocod_kernel_local_step_host_noalloc(dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(),
                                                  host.data_ptr(), n, 0.1, 0.9, 0.0, None)
    assert rc == E.ERR_TOO_LARGE
    assert b"capacity" in lib.cocod_strerror(rc)
    assert lib.cocod_kernel_local_step_host_noalloc(None, None, None, None, 8, 0.1, 0.9, 0.0, None) == E.ERR_INVALID
    # exactly at the limit is accepted
    m = E.NOALLOC_MAX_ELEMS
    x, v = torch.zeros(m, device="cuda"), torch.zeros(m, device="cuda")
    g = torch.ones(m).pin_memory()
    E.kernel_local_step_host_noalloc(x, x, v, g, 0.5, 0.0, 0.0)
    torch.cuda.synchronize()
    assert torch.all(x == -0.5) and torch.all(v == 1.0)
