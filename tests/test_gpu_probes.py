"""The two machine-rate probes: they run, count what they say they count, and reject bad layouts."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fo():
    import paper_1801_00829_b200 as m
    m.load_library()
    return m


def test_gather_probe_reads_the_rows_it_is_given(fo):
    import torch
    dev = torch.device("cuda", 0)
    rows, cols, n = 5000, 100, 200_003
    V = torch.arange(rows * cols, dtype=torch.float64, device=dev).reshape(rows, cols) % 1024
    g = torch.Generator(device=dev)
    g.manual_seed(3)
    idx = torch.randint(0, rows, (n,), generator=g, device=dev, dtype=torch.int32)
    out = torch.zeros(fo.probe_out_len(), dtype=torch.float64, device=dev)
    moved = fo.probe_l2_gather(V, idx, out)
    torch.cuda.synchronize()
    assert moved == n * cols * 8
    # every gathered element is added exactly once somewhere in `out` (small integers: exact);
    # the last group of four repeats its first row for the missing ones
    want = V[idx.long()].sum().item()
    pad = (-n) % 4
    want += pad * V[idx[n - (n % 4)].long()].sum().item() if pad else 0.0
    assert out.sum().item() == want


def test_gather_probe_rejects_odd_or_unaligned(fo):
    import torch
    from paper_1801_00829_b200.binding import FusedOpsError
    dev = torch.device("cuda", 0)
    idx = torch.zeros(8, dtype=torch.int32, device=dev)
    with pytest.raises(FusedOpsError):
        fo.probe_l2_gather(torch.zeros((4, 7), dtype=torch.float64, device=dev), idx)
    base = torch.zeros(4 * 8 + 1, dtype=torch.float64, device=dev)
    with pytest.raises(FusedOpsError):
        fo.probe_l2_gather(base[1:].reshape(4, 8), idx)


def test_fma_probe_counts_flops_and_converges(fo):
    import torch
    dev = torch.device("cuda", 0)
    out = torch.zeros(fo.probe_out_len(), dtype=torch.float64, device=dev)
    flops = fo.probe_fp64_fma(4000, out)
    torch.cuda.synchronize()
    assert flops == 16 * 4000 * fo.probe_out_len()
    # x <- 0.999999 x + 1e-6 moves every chain towards its fixed point 1.0 from below
    got = out.cpu().numpy()
    assert np.all(np.isfinite(got)) and np.all(got > 0.0) and np.all(got < 8.0)


def test_bulk_gather_probe_lands_the_rows_it_is_given(fo):
    import torch
    dev = torch.device("cuda", 0)
    rows, cols, n = 5000, 100, 200_003
    V = torch.arange(rows * cols, dtype=torch.float64, device=dev).reshape(rows, cols) % 1024
    g = torch.Generator(device=dev)
    g.manual_seed(5)
    idx = torch.randint(0, rows, (n,), generator=g, device=dev, dtype=torch.int32)
    out = torch.full((fo.probe_out_len(),), 7.0, dtype=torch.float64, device=dev)
    moved = fo.probe_bulk_gather(V, idx, out)
    torch.cuda.synchronize()
    assert moved == n * cols * 8
    flag = fo.probe_bulk_flag_index()
    assert out[flag].item() == 0.0                       # no bounded wait ran out
    # every lane adds, per batch of 16 rows, element (lane mod cols) of the batch's first row
    first = V[idx[::16].long()][:, :32].sum().item()
    assert out[:flag].sum().item() == first


def test_bulk_gather_probe_rejects_odd_or_unaligned(fo):
    import torch
    from paper_1801_00829_b200.binding import FusedOpsError
    dev = torch.device("cuda", 0)
    idx = torch.zeros(8, dtype=torch.int32, device=dev)
    with pytest.raises(FusedOpsError):
        fo.probe_bulk_gather(torch.zeros((4, 7), dtype=torch.float64, device=dev), idx)
    base = torch.zeros(4 * 8 + 1, dtype=torch.float64, device=dev)
    with pytest.raises(FusedOpsError):
        fo.probe_bulk_gather(base[1:].reshape(4, 8), idx)
