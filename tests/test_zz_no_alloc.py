"""Allocation-free weight gradient (lp_weight_grad_static) against the ordinary entry point.

Who needs it: callers that cannot call cudaMalloc when the gradient is due -- loops that ban
allocator calls because they lock the driver and may synchronise the device, processes that gave
all device memory to a pool at start-up, code sections where the runtime refuses to allocate.  The entry point keeps its
partial sums in a fixed array inside the library, so this test also checks that a second call, which
finds the first call's data in that array, still returns the right answer.

The file sorts last on purpose: a run that stops at the first failure has then run every other test.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def pkg():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import __graft_entry__ as ge
    ge.build()
    import paper_2506_20818_b200 as p
    return p


def rel_l2(a, b):
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def test_static_weight_grad_matches_ordinary_entry_twice(pkg):
    import workloads as wl
    g = wl.erdos_renyi(50, 100, seed=0)
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, None, wl.node_features(g.n, 8, 0))
    rng = np.random.default_rng(5)
    # two calls in a row with different shapes: the second finds the first one's partial sums in the array
    for M, K, N in ((70001, 256, 128), (3000, 512, 256)):
        A = torch.from_numpy(rng.standard_normal((M, K)).astype(np.float32)).to(DEV)
        dZ = torch.from_numpy(rng.standard_normal((M, N)).astype(np.float32)).to(DEV)
        want = ctx.op_weight_grad(A, dZ)
        got = pkg.weight_grad_static(A, dZ)
        torch.cuda.synchronize()
        assert rel_l2(got.cpu().numpy(), want.cpu().numpy()) < 1e-5  # FP32-path tolerance of the parity tests
        exact = A.double().T @ dZ.double()
        assert rel_l2(got.double().cpu().numpy(), exact.cpu().numpy()) < 1e-5
    # same inputs again: the result is reproducible bit for bit, and the call takes no device memory: the free
    # memory of the device is the same before and after it (the output tensor is allocated beforehand)
    import ctypes as C
    lib = pkg.load_library()
    again = torch.empty_like(got)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    rc = lib.lp_weight_grad_static(C.c_int32(0), C.c_void_p(torch.cuda.current_stream().cuda_stream), C.c_int64(A.shape[0]), C.c_int32(dZ.shape[1]),
                                   C.c_int32(A.shape[1]), C.c_void_p(A.data_ptr()), C.c_void_p(dZ.data_ptr()), C.c_void_p(again.data_ptr()))
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert rc == 0 and free_after == free_before
    assert torch.equal(again, got)
    ctx.close()


def test_static_weight_grad_at_the_size_limit(pkg):
    # K * N = 2^21 exactly: the fixed array holds one partial tile, so the rows are not split at all
    import workloads as wl
    g = wl.erdos_renyi(50, 100, seed=0)
    ctx = pkg.Context(0)
    ctx.load_graph(g.n, g.rowptr, g.col, None, wl.node_features(g.n, 8, 0))
    rng = np.random.default_rng(6)
    A = torch.from_numpy(rng.standard_normal((37, 2048)).astype(np.float32)).to(DEV)
    dZ = torch.from_numpy(rng.standard_normal((37, 1024)).astype(np.float32)).to(DEV)
    for _ in range(2):
        got = pkg.weight_grad_static(A, dZ)
        torch.cuda.synchronize()
        assert rel_l2(got.double().cpu().numpy(), (A.double().T @ dZ.double()).cpu().numpy()) < 1e-5
    assert rel_l2(got.cpu().numpy(), ctx.op_weight_grad(A, dZ).cpu().numpy()) < 1e-5
    ctx.close()


def test_static_weight_grad_rejects_oversize(pkg):
    A = torch.zeros((4, 2048), device=DEV)
    dZ = torch.zeros((4, 2048), device=DEV)  # K * N = 2^22 > 2^21
    with pytest.raises(pkg.LpError) as ei:
        pkg.weight_grad_static(A, dZ)
    assert ei.value.status == -1 and "exceeds" in str(ei.value)
