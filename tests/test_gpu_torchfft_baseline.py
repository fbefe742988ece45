"""The torch.fft comparator that bench.py times beside the library computes the same operator: its coefficients and
its reconstruction agree with the library's on the paper's principal layout (fp32 on both sides)."""
import numpy as np
import pytest

import workloads as wl
from helpers import library_plan

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def test_comparator_matches_library_on_table1_layout():
    from torchfft_baseline import TorchFftCqt
    w = wl.scaled(wl.CONFIGS["table1"], channels=3)
    plan = library_plan(w)
    tf = TorchFftCqt(plan, torch.device("cuda"))
    x = torch.from_numpy(wl.make_signal(w)).cuda()
    c_lib = plan.analyse(x, valid_len=w.valid_len)
    c_tf = tf.analyse(x)
    o = 0
    for bi in plan.bands():
        a, b = c_tf[:, o:o + bi.M], c_lib[:, o:o + bi.M]
        rel = (torch.linalg.norm(a - b, dim=-1) / torch.linalg.norm(b, dim=-1)).max().item()
        assert rel <= 2e-5, (bi.centre_bin, rel)
        o += bi.M
    y_lib = plan.synthesise(c_lib, valid_len=w.valid_len)
    y_tf = tf.synthesise(c_lib)
    assert (torch.linalg.norm(y_tf - y_lib, dim=-1) / torch.linalg.norm(y_lib, dim=-1)).max().item() <= 2e-5
    plan.close()
