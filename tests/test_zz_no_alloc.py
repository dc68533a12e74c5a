"""The entry point that allocates nothing (collected last on purpose).

Some users of this library may not call cudaMalloc at all: a plugin living inside an
application that owns every byte of device memory, or a loop that must stay away from the
allocator once it is running.  For them si_ffn_forward_noalloc keeps its scratch in a fixed
array inside the library.  This test calls it through the C ABI twice in a row -- the second
call finds the first call's leftovers in the shared scratch -- and checks each result against
the ordinary entry point on the same inputs.
"""
import numpy as np
import pytest
import torch

from paper_2607_18081_b200 import workloads as wl
from tests.gpu_utils import LoadedModel, assert_close, from_dev, to_dev

pytestmark = pytest.mark.gpu


def test_noalloc_entry_point_matches_the_ordinary_one_twice_in_a_row():
    from paper_2607_18081_b200 import api
    cfg = wl.CONFIGS["c1"]
    m = LoadedModel(cfg)
    k = cfg.k_active
    lists = wl.zipf_lists(cfg, 0, 2, slot_of_rank=m.slot_of_rank[0], first_token=300)
    x = wl.x_tokens(cfg, 0, 2, first_token=300)
    ws = m.store.workspace(1, k, 1)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # Set-up call: the first call on a device looks up the scratch array's address, and the CUDA
    # runtime loads the library image (the array included) on first use.  Free memory is compared
    # only around later calls.
    warm = torch.empty(cfg.d_model, dtype=torch.float32, device="cuda")
    api.si_ffn_forward_noalloc(m.store.handle, 0, to_dev(x[0], cfg.dtype), torch.from_numpy(lists[0]).cuda(), k,
                               warm, 0, status)
    torch.cuda.synchronize()
    for call in range(2):                      # two calls in a row share the built-in scratch
        xd = to_dev(x[call], cfg.dtype)
        idx = torch.from_numpy(lists[call]).cuda()
        for flags in (0, api.SI_FLAG_RESIDUAL):
            y_new = torch.empty(cfg.d_model, dtype=torch.float32, device="cuda")
            y_same_kernels = torch.empty_like(y_new)
            y_default = torch.empty_like(y_new)
            # nothing may be allocated by the call: torch's own allocator must not have moved, and the device's free
            # memory must be what it was (another process on the GPU can change the latter: look twice before failing)
            for attempt in range(2):
                free_before, torch_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_reserved()
                api.si_ffn_forward_noalloc(m.store.handle, 0, xd, idx, k, y_new, flags, status)
                torch.cuda.synchronize()
                assert torch.cuda.memory_reserved() == torch_before
                if torch.cuda.mem_get_info()[0] == free_before:
                    break
            else:
                raise AssertionError("free device memory changed around the call that allocates nothing")
            api.si_ffn_forward(m.store.handle, 0, xd, 1, idx, None, k, y_same_kernels,
                               flags | api.SI_FLAG_SIMPLE_KERNELS, ws, status)
            api.si_ffn_forward(m.store.handle, 0, xd, 1, idx, None, k, y_default, flags, ws, status)
            torch.cuda.synchronize()
            assert status.item() == 0
            # same kernels, same order of sums: identical bits
            assert torch.equal(y_new, y_same_kernels)
            # the default (persistent) path sums in another order: within the parity tolerance
            assert_close(from_dev(y_new), from_dev(y_default).astype(np.float64), f"call {call} flags {flags}")
            ref = m.oracle_y(0, x[call], lists[call])
            if flags:
                ref = ref + wl.bits_to_float64(x[call], cfg.dtype)
            assert_close(from_dev(y_new), ref, f"call {call} flags {flags} vs oracle")
    # another device current than the store's: refused on the host (only where there is a second device to make current)
    if torch.cuda.device_count() > 1:
        with torch.cuda.device(1):
            with pytest.raises(api.SelectInferError) as e:
                api.si_ffn_forward_noalloc(m.store.handle, 0, to_dev(x[0], cfg.dtype), torch.from_numpy(lists[0]).cuda(0), k,
                                           torch.empty(cfg.d_model, dtype=torch.float32, device="cuda:0"), 0)
            assert e.value.status == api.SI_ERR_INVALID_ARG
    # bf16 output variant is not available for an fp16 store, and sizes are checked
    with pytest.raises(api.SelectInferError) as e:
        api.si_ffn_forward_noalloc(m.store.handle, 0, to_dev(x[0], cfg.dtype), torch.from_numpy(lists[0]).cuda(),
                                   cfg.n_loaded + 1, torch.empty(cfg.d_model, dtype=torch.float32, device="cuda"), 0)
    assert e.value.status == api.SI_ERR_OUT_OF_RANGE
