"""Plans used from several host threads at once, each with its own stream: the library's process-wide state (launch
counter, per-device grants of shared memory, the SM count) must hold, and the results must be the bits of a
single-threaded run (every kernel adds in a fixed order)."""
import threading

import pytest
import torch

from oracle import psattn_oracle as orc
from paper_2106_09236_b200 import binding as ps
from test_parity_gpu import _dev, _synth

pytestmark = pytest.mark.gpu

CASES = {"fused": (4, 8, 1024, 1), "staged": (2, 8, 3000, 2), "short": (16, 4, 300, 3)}


def _work(name, out, repeats):
    B, H, T, seed = CASES[name]
    c = 5.0
    n_cols = max(orc.count(c, L) for L in range(1, T + 1))
    inp = _synth(B, H, T, seed, n_cols, "bf16", None)
    dev, tdt = _dev(inp, "bf16")
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=n_cols)
        kept = []
        for it in range(repeats):
            O, sel = plan.psattn_forward(dev["Q"], dev["K"], dev["V"], dev["lengths"], dev["sample_idx"])
            if it % 25 == 0:
                kept.append((O.clone(), sel.clone()))
        st.synchronize()
        same = all(torch.equal(kept[0][0], o) and torch.equal(kept[0][1], s) for o, s in kept)
        out[name] = (same and plan.psattn_read_status() == 0, kept[0][0].cpu(), kept[0][1].cpu())
        plan.close()


def test_three_threads_with_their_own_plans_and_streams():
    together, alone = {}, {}
    threads = [threading.Thread(target=_work, args=(name, together, 100)) for name in CASES]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    for name in CASES:
        _work(name, alone, 26)
    for name in CASES:
        assert together[name][0] and alone[name][0], name
        assert torch.equal(together[name][1], alone[name][1]) and torch.equal(together[name][2], alone[name][2]), name
