"""pat_project_static: the projection entry point that uses the library's built-in scratch array.

It serves callers that cannot allocate device memory where they run (all memory reserved by a pool at start-up,
plug-ins inside another allocator, loops that must not trigger an allocation's device-wide synchronisation).
The file is named so that pytest collects it last: a run that stops at the first failure has then already
run every other test.
"""
import gc

import numpy as np
import pytest
import torch

import oracle
import paper_2001_07710_b200 as pc
from paper_2001_07710_b200 import workloads

pytestmark = pytest.mark.gpu


def _run_both(seed, F, C, K, n_keep):
    w_np = workloads.make_weights(np.random.default_rng(seed), F, C)
    w = torch.from_numpy(w_np).cuda()
    masks = pc.pat_library_builtin(K)
    # reference: the ordinary entry point with a caller-provided workspace
    pid_ref, wm_ref = pc.pat_project(w, masks, n_keep)
    torch.cuda.synchronize()
    # outputs are preallocated here, before the call: the call itself must allocate nothing
    pid = torch.full((F, C), 0x5A, dtype=torch.uint8, device="cuda")
    wm = torch.full((F, C, 3, 3), float("nan"), dtype=torch.float32, device="cuda")
    # a first call on this device looks up the scratch array's address (and loads the module); the calls that are
    # measured come after it
    pc.pat_project_static(w, masks, n_keep, pid, wm)
    pid.fill_(0x5A)
    wm.fill_(float("nan"))
    gc.collect()                                    # tensors that earlier tests left in reference cycles go now, not inside the window
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()          # torch's allocator ...
    torch.cuda.reset_peak_memory_stats()            # ... and its high-water mark from here on
    free_before = torch.cuda.mem_get_info()[0]      # the driver's view (cudaMemGetInfo): sees any cudaMalloc
    pc.pat_project_static(w, masks, n_keep, pid, wm)
    torch.cuda.synchronize()
    assert torch.cuda.max_memory_allocated() == before and torch.cuda.memory_allocated() <= before
    assert torch.cuda.mem_get_info()[0] == free_before
    assert pc.pat_query_status() == 0
    # against the oracle (brute force over the library, sort for connectivity): bit for bit
    pid_o, wm_o, _ = oracle.project(w_np, masks, n_keep)
    assert np.array_equal(pid.cpu().numpy(), pid_o)
    assert np.array_equal(wm.cpu().numpy().view(np.uint32), wm_o.view(np.uint32))
    # integer and bit-pattern work: the tolerance of the projection tests is exact equality
    assert torch.equal(pid, pid_ref)
    assert torch.equal(wm.view(torch.int32), wm_ref.view(torch.int32))
    assert int((pid != 255).sum()) == n_keep


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    # two calls in a row on different layers: the second one finds the first one's leftovers in the scratch array
    _run_both(1, 256, 256, 8, 256 * 256 // 8)
    _run_both(2, 64, 96, 12, 64 * 96 * 3 // 10)
    # and once more on the first shape with other data (ties and thresholds differ)
    _run_both(3, 256, 256, 4, 256 * 256 // 2)


def test_static_scratch_rejects_layers_beyond_its_size():
    limit = pc.pat_project_static_max_kernels()
    assert limit == 262144
    F, C = 1024, 512                                              # 524288 kernels: twice the limit
    w = torch.zeros((F, C, 3, 3), device="cuda")
    pid = torch.zeros((F, C), dtype=torch.uint8, device="cuda")
    with pytest.raises(pc.PatError) as e:
        pc.pat_project_static(w, pc.pat_library_builtin(8), 10, pid, torch.empty_like(w))
    assert e.value.code == 8 and "exceeds" in str(e.value)
    assert not pid.any()                                          # nothing ran
