"""The allocation-free count entry point (retexo_cross_partition_bytes_static), for callers
that may not call cudaMalloc: it must give exactly what the workspace-taking entry point
gives, on two calls in a row (its built-in scratch keeps the previous call's contents), and
it must refuse problems larger than that scratch.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2302_13053_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_static_scratch_entry_point_matches_the_workspace_one_twice_in_a_row():
    from paper_2302_13053_b200 import binding as B
    cases = []
    w = wl.make_config(4, scale=0.02)                      # 1000 partitions: shared-memory bitmap path
    cases.append((w.rowptr, w.colidx, w.part, w.n_parts, [602, 256, 256]))
    w = wl.make_config(2)                                  # 100 partitions
    cases.append((w.rowptr, w.colidx, w.part, w.n_parts, [500, 128, 128]))
    w = wl.make_config(3)                                  # node-level: the many-partition kernels and their lists
    cases.append((w.rowptr, w.colidx, w.part, w.n_parts, [128, 64]))
    for rowptr, colidx, part, n_parts, dims in cases:
        rp, ci, pt = dev(rowptr.astype(np.int64)), dev(colidx.astype(np.int32)), dev(part.astype(np.int32))
        ref = B.retexo_cross_partition_bytes(rp, ci, pt, n_parts, dims, 4, per_part=False)
        out = torch.zeros(3 + len(dims), dtype=torch.int64, device="cuda")
        for call in range(2):
            out.fill_(-1)
            B.retexo_cross_partition_bytes_static(rp, ci, pt, n_parts, dims, out)
            torch.cuda.synchronize()
            got = out.cpu().numpy().view(np.uint64)
            assert int(got[0]) == ref["cross_edges"], call
            assert int(got[1]) == ref["boundary_pairs"], call
            assert int(got[2]) == ref["bytes_total"], call
            np.testing.assert_array_equal(got[3:3 + len(dims)], ref["bytes_per_round"])
        # what the entry point exists for: a further call takes no device memory, neither from the
        # driver (free bytes of the device unchanged) nor through torch's allocator
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        held_before = torch.cuda.memory_allocated()
        B.retexo_cross_partition_bytes_static(rp, ci, pt, n_parts, dims, out)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.cuda.memory_allocated() == held_before


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    from paper_2302_13053_b200 import binding as B
    limit = B.lib().retexo_cross_partition_static_scratch_bytes()
    assert limit == 4 << 20
    n = 3_000_000                                           # node-level partition of 3 M nodes needs > 4 MiB of lists
    rp = torch.zeros(n + 1, dtype=torch.int64, device="cuda")
    ci = torch.zeros(1, dtype=torch.int32, device="cuda")[:0]
    pt = torch.zeros(n, dtype=torch.int32, device="cuda")
    out = torch.zeros(4, dtype=torch.int64, device="cuda")
    with pytest.raises(B.RetexoError, match="not supported"):
        B.retexo_cross_partition_bytes_static(rp, ci, pt, n, [4], out)
