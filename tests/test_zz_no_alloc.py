"""hap_argmin_static: the argmin entry point for callers that cannot allocate device memory
(processes whose GPU memory is already owned by a framework allocator or a start-up arena).
It must give exactly what hap_argmin gives, on consecutive calls that share its built-in scratch."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def test_static_argmin_matches_hap_argmin_on_two_calls_in_a_row():
    import paper_2609_39350_b200 as hap
    from paper_2609_39350_b200.build import build_library
    from gen import problems
    build_library()
    assert torch.cuda.is_available()
    hp = hap.hap_problem_create(problems.tiny())
    hap.hap_enumerate(hp)
    g = torch.Generator(device="cuda").manual_seed(7)
    # first call: several blocks of partials and a ragged tail; the minimum occurs twice (lowest index wins)
    a = torch.randint(10, 1 << 40, (3 * 16384 + 777,), dtype=torch.int64, device="cuda", generator=g)
    a[40000] = 5
    a[1234] = 5
    # second call: shorter input, so partial slots written by the first call stay behind in the scratch
    b = torch.randint(10, 1 << 40, (16384 + 5,), dtype=torch.int64, device="cuda", generator=g)
    b[-1] = 3
    out = torch.empty(2, dtype=torch.int64, device="cuda")          # caller-owned output, reused
    hap.hap_argmin_static(b, out=out)        # the first call on a device looks up the scratch address
    torch.cuda.synchronize()
    for x in (a, b, a):
        ref = hap.hap_argmin(hp, x)
        torch.cuda.synchronize()
        # with a caller-owned output the call must leave the device's memory as it is: nothing allocated through
        # torch, nothing taken from the driver
        free0, used0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        got = hap.hap_argmin_static(x, out=out)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == used0 and torch.cuda.mem_get_info()[0] == free0
        assert got.cpu().tolist() == ref.cpu().tolist()
        assert got.cpu().tolist() == [int(x.min()), int(torch.nonzero(x == x.min())[0])]
    # all-infeasible input keeps the library's convention for "nothing found"
    inf = torch.full((100,), hap.INF, dtype=torch.int64, device="cuda")
    assert hap.hap_argmin_static(inf, out=out).cpu().tolist() == hap.hap_argmin(hp, inf).cpu().tolist()
    # sizes outside [1, 2^26] (and beyond the tensor) are refused before anything is launched; so are tensors that
    # are not contiguous int64
    with pytest.raises(hap.HapError):
        hap.hap_argmin_static(a[::2], out=out)
    with pytest.raises(hap.HapError):
        hap.hap_argmin_static(a.to(torch.int32), out=out)
    for bad in (0, a.numel() + 1, (1 << 26) + 1):
        with pytest.raises(hap.HapError) as e:
            hap.hap_argmin_static(a, out=out, count=bad)
        assert e.value.name == "HAP_E_RANGE"
    # the library's own limit (2^26 costs), asked directly: refused with HAP_E_RANGE, nothing read or launched
    import ctypes as C
    st = hap.load_library().hap_argmin_static(C.c_void_p(a.data_ptr()), C.c_uint64((1 << 26) + 1), C.c_void_p(out.data_ptr()),
                                              C.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert st == 4
    torch.cuda.synchronize()
    assert out.cpu().tolist() == hap.hap_argmin(hp, inf).cpu().tolist()      # the refused calls wrote nothing
    hap.hap_problem_destroy(hp)
