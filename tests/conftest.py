import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def tiny_cfg(**over):
    """A hand-sized model for brute-force checks."""
    from paper_2507_23777_b200 import inputs
    c = inputs.config(0)
    c.update(name="unit", n_layers=2, d_model=32, n_heads=2, d_head=16, d_ff=64, n_cond=5, d_cond=32,
             vocab=50, n_draft=2, head_hidden=32, page_size=4, max_seq_len=64, seed=11, sigma=0.3)
    c.update(over)
    return c


def gpu_cfg(**over):
    """The smallest model the CUDA library accepts (d_model and d_ff multiples of 128, d_head 32, 32-token
    pages) with ragged sizes everywhere else: 50-token vocabulary, 5 condition latents of width 64."""
    c = tiny_cfg(d_model=128, n_heads=4, d_head=32, d_ff=256, n_cond=5, d_cond=64, head_hidden=128, page_size=32,
                 max_seq_len=96)
    c.update(over)
    return c


@pytest.fixture(scope="session")
def oracle_mod():
    import oracle
    oracle.build()
    return oracle
