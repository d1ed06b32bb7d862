"""The allocation-free probe entry point (chimera_probes_static) against the workspace-based probe stage.

Some users of the library may not allocate device memory at query time (serving loops that fix memory at start-up;
processes where another component owns the memory pool).  chimera_probes_static serves them with scratch that is built
into the library image.  This test calls it through the C ABI twice in a row (the scratch is shared between calls and
keeps its contents, so the second call runs on a dirty array) and requires the same probes, bit for bit, as stage 2 of
chimera_run_stages on the same score table.  It is collected last so that a run stopping at the first failure has
already run every other test; it passes alone in a fresh process as well.
"""
import numpy as np
import pytest
import torch

from helpers import random_corpus, unit_rows

pytestmark = pytest.mark.gpu


def _case(pkg, seed, K, N, D, nq, B, nprobe):
    cent, cids, codes, doclens = random_corpus(seed, N, K, D, 2, len_lo=1, len_hi=20)
    dev = torch.device("cuda:0")
    gix = pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev), torch.from_numpy(codes).to(dev),
                    torch.from_numpy(doclens).to(dev), 2)
    rng = np.random.default_rng(seed)
    q = torch.from_numpy(np.stack([unit_rows(rng, nq, D) for _ in range(B)])).to(dev)
    taps = gix.alloc_taps(B, nq, nprobe, 8)
    gix.run_stages(1, 2, q, B, nq, nprobe, 8, 4, taps)        # existing entry point: table and probes
    torch.cuda.synchronize()
    return taps.score_table.clone(), taps.probes.clone()


def test_static_probes_match_workspace_probes_on_two_calls_in_a_row():
    import paper_2608_23553_b200 as pkg
    # two different problems back to back: the second call finds the first call's partial lists in the shared array
    table_a, probes_a = _case(pkg, 31, K=3000, N=300, D=64, nq=32, B=3, nprobe=4)
    table_b, probes_b = _case(pkg, 32, K=700, N=200, D=32, nq=40, B=2, nprobe=9)
    got_a = pkg.probes_static(table_a, 4)
    got_b = pkg.probes_static(table_b, 9)
    got_a2 = pkg.probes_static(table_a, 4)
    torch.cuda.synchronize()
    assert torch.equal(got_a, probes_a)
    assert torch.equal(got_b, probes_b)
    assert torch.equal(got_a2, probes_a)


def test_static_probes_allocate_no_device_memory():
    """What the entry point exists for: after one warm-up call (which may load the library's kernels and look the
    built-in array up), a call straight through the C ABI with a caller-owned output buffer leaves the device's free
    memory and torch's own allocation count exactly where they were."""
    import ctypes
    import paper_2608_23553_b200 as pkg
    table, probes = _case(pkg, 33, K=1500, N=100, D=32, nq=32, B=2, nprobe=4)
    out = torch.empty_like(probes)
    L = pkg.lib()
    args = (ctypes.c_void_p(table.data_ptr()), ctypes.c_int64(table.shape[1]), ctypes.c_int32(table.shape[0]),
            ctypes.c_int32(table.shape[2]), ctypes.c_int32(4), ctypes.c_void_p(torch.cuda.current_stream().cuda_stream),
            ctypes.c_void_p(out.data_ptr()))
    assert L.chimera_probes_static(*args) == 0                   # warm-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    torch0 = torch.cuda.memory_allocated()
    for _ in range(3):
        assert L.chimera_probes_static(*args) == 0
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    # (free memory is device-wide: it must not have gone down; torch's own count must not have moved at all)
    assert free1 >= free0 and torch.cuda.memory_allocated() == torch0
    assert torch.equal(out, probes)


def test_static_probes_reject_sizes_beyond_the_built_in_array():
    import paper_2608_23553_b200 as pkg
    # 64 queries x 10 lists x nprobe 64 x q_len 120 x 8 B is far beyond 4 MiB
    table = torch.zeros(64, 4096, 120, dtype=torch.int32, device="cuda:0")
    with pytest.raises(pkg.ChimeraError) as e:
        pkg.probes_static(table, 64)
    assert e.value.code == 3
    with pytest.raises(pkg.ChimeraError) as e:
        pkg.probes_static(table[:1, :8].contiguous(), 9)       # nprobe > n_centroids
    assert e.value.code == 1
