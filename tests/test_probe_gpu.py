"""The gather microbenchmarks behind the `roofline_gather` ceilings: every mode launches, stays inside its buffers
(small buffers, so any stray index would show) and rejects bad arguments.  No timing here."""
import pytest
import torch

from paper_2106_09236_b200 import binding as ps

pytestmark = pytest.mark.gpu


def test_every_mode_runs_on_a_small_buffer():
    sink = torch.zeros(4, dtype=torch.int32, device="cuda")
    rows = torch.randn(1024 * 32, device="cuda")                # 1024 rows of 128 bytes
    for mode, warps, rounds in ((0, 16, 64), (1, 24, 64), (2, 24, 64), (3, 16, 64), (6, 16, 64), (8, 16, 64), (11, 24, 64),
                                (12, 24, 64), (12, 6, 8)):
        n = ps.psattn_probe_gather(mode, rows if mode in (1, 2, 11, 12) else None, 8, warps, rounds, sink)
        torch.cuda.synchronize()
        assert n > 0
    assert sink.cpu().tolist()[1] == 0                          # no bounded wait of the bulk-copy modes ran out
    # the mixed mode counts half as many rounds for every sixth warp
    assert ps.psattn_probe_gather(12, rows, 2, 12, 8, sink) == 2 * (10 * 8 + 2 * 4) * 16
    torch.cuda.synchronize()


def test_bucketed_chunk_loop_counts_its_pairs():
    lib = ps.load()
    sink = torch.zeros(4, dtype=torch.int32, device="cuda")
    rows = torch.randn(8192 * 32, device="cuda")                # 8192 rows of 128 bytes
    for mode in (13, 14):
        sink.zero_()
        assert lib.psattn_probe_gather(mode, rows.data_ptr(), 8192, 4, 16, 2, sink.data_ptr(), None) == 0
        torch.cuda.synchronize()
        pairs = int(sink[2:4].view(torch.int64).item())
        cells = 4 * 2 * 2048                                    # CTAs x work items x queries
        assert 5.0 < pairs / cells < 6.5                        # the mean of Binomial(46, 1/8) is 5.75
    assert lib.psattn_probe_gather(13, rows.data_ptr(), 1024, 4, 16, 2, sink.data_ptr(), None) == 2     # buffer too small
    assert lib.psattn_probe_gather(13, rows.data_ptr(), 8192, 4, 8, 2, sink.data_ptr(), None) == 2      # 16 warps only


def test_bad_arguments_are_refused():
    lib = ps.load()
    sink = torch.zeros(4, dtype=torch.int32, device="cuda")
    rows = torch.randn(1024 * 32, device="cuda")
    assert lib.psattn_probe_gather(1, None, 1024, 8, 24, 64, sink.data_ptr(), None) == 1            # no buffer
    assert lib.psattn_probe_gather(11, rows.data_ptr(), 1024, 8, 25, 64, sink.data_ptr(), None) == 2     # too many warps
    assert lib.psattn_probe_gather(11, rows.data_ptr() + 4, 1023, 8, 24, 64, sink.data_ptr(), None) == 5   # misaligned
    assert lib.psattn_probe_gather(99, rows.data_ptr(), 1024, 8, 24, 64, sink.data_ptr(), None) == 2
