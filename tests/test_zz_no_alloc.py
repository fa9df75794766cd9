"""The allocation-free forward entry point (collected last on purpose).

fewbit_fwd_host_static is for callers that cannot allocate device memory where
they need the forward pass (their process's pool owns the device, they run
under a fixed budget, or they cannot risk the synchronisation an allocation
may cause): its device staging area is a fixed array inside the library.  The
test calls it through the C ABI twice in a row with different inputs -- the
array keeps the first call's data, which must not leak into the second -- and
compares every output byte with what the ordinary host entry point returns
and with the oracle.  It also checks what the entry point is for: once the
first call on the device has been made, a call changes neither the free device
memory nor launches anything but its one kernel.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2202_00441_b200 as fb
from paper_2202_00441_b200 import workloads as wl
from helpers import finite_mask, ulp_distance

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_static_entry_point_matches_the_workspace_entry_point_twice_in_a_row(dtype):
    dev = torch.device("cuda", 0)
    cap = fb.fewbit_static_max_elements()
    assert cap == 262144
    gen = torch.Generator().manual_seed(77)
    calls = [("gelu", 4, cap), ("silu", 3, 100000 + 19), ("tanh", 1, 1), ("gelu", 4, 4099)]
    for act, bits, n in calls:
        t = fb.fewbit_table_create(act, bits)
        x = (torch.randn(n, generator=gen) * 2).to(dtype)
        words = fb.fewbit_packed_bytes(n, bits) // 4
        # reference: the existing entry point with a caller-owned device workspace
        y_ref, p_ref = torch.empty_like(x), torch.empty(words, dtype=torch.int32)
        ws = torch.empty(fb.fewbit_host_workspace_bytes(n, dtype, bits), dtype=torch.uint8, device=dev)
        fb.fewbit_fwd_host(t, x, y_ref, p_ref, ws)
        # the allocation-free call; outputs pre-filled so that untouched bytes would show
        y, p = torch.full_like(x, 3.0), torch.full((words,), 0x55555555, dtype=torch.int32)
        fb.fewbit_fwd_host_static(t, x, y, p, device=dev)
        assert np.array_equal(wl.to_numpy_bits(y), wl.to_numpy_bits(y_ref)), (act, bits, n)   # same kernel: tolerance 0
        assert np.array_equal(p.numpy(), p_ref.numpy()), (act, bits, n)
        # and against the oracle: codes bit-exact, y within 2 ulp
        s, _ = t.arrays()
        xn = wl.to_numpy_bits(x)
        y_or, p_or = oracle.fwd(act, bits, s, xn)
        assert np.array_equal(p.numpy().view(np.uint32), p_or), (act, bits, n)
        ok = finite_mask(xn)
        assert ulp_distance(wl.to_numpy_bits(y)[ok], y_or[ok]).max() <= 2, (act, bits, n)


def test_static_entry_point_allocates_nothing_and_launches_one_kernel():
    dev = torch.device("cuda", 0)
    t = fb.fewbit_table_create("silu", 4)
    n = 200000 + 3
    x = torch.randn(n).bfloat16().pin_memory()
    y = torch.empty_like(x).pin_memory()
    p = torch.empty(fb.fewbit_packed_bytes(n, 4) // 4, dtype=torch.int32).pin_memory()
    fb.fewbit_fwd_host_static(t, x, y, p, device=dev)        # the set-up call: loads the module that holds the array
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info(dev)
    launches_before = fb.fewbit_launch_count()
    for _ in range(3):
        fb.fewbit_fwd_host_static(t, x, y, p, device=dev)
    free_after, _ = torch.cuda.mem_get_info(dev)
    assert free_after == free_before
    assert fb.fewbit_launch_count() - launches_before == 3


def test_static_entry_point_rejects_oversize_and_bad_arguments():
    t = fb.fewbit_table_create("gelu", 2)
    n = fb.fewbit_static_max_elements() + 1
    x = torch.zeros(n)
    y = torch.empty_like(x)
    p = torch.empty(fb.fewbit_packed_bytes(n, 2) // 4, dtype=torch.int32)
    with pytest.raises(fb.FewbitError) as e:
        fb.fewbit_fwd_host_static(t, x, y, p, device="cuda:0")
    assert e.value.status == 6 and "fixed staging area" in str(e.value)
    lib = fb.load_library()
    assert lib.fewbit_fwd_host_static(None, x.data_ptr(), y.data_ptr(), p.data_ptr(), 10, 0, None) == 1
    assert lib.fewbit_fwd_host_static(t.handle, None, y.data_ptr(), p.data_ptr(), 10, 0, None) == 1
    assert lib.fewbit_fwd_host_static(t.handle, None, None, None, 0, 0, None) == 0
