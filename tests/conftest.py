import os
import sys
from pathlib import Path

import numpy as np
import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def tiny_case():
    """Tiny config: d=64, one KV head, 4 query heads, S=1024, Lloyd 10 iterations."""
    from paper_2608_04074_b200 import synth, workloads
    from oracle import novakv_oracle as O

    wl = workloads.tiny()
    laws = wl.laws()
    cal = wl.calibration(laws)
    k, v = synth.draw_kv(laws, 1000 * wl.seed + 11, int(wl.seq_lens[0]))
    q = synth.draw_q(laws, 1000 * wl.seed + 12, 1)[0]
    k = synth.to_bf16_representable(k)
    v = synth.to_bf16_representable(v)
    q = synth.to_bf16_representable(q)
    return dict(wl=wl, laws=laws, cal=cal, oracle=O.Oracle.from_calibration(cal), k=k, v=v, q=q)


def has_cuda() -> bool:
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False
