"""Seeded sweep over random batch shapes -- batch size, vocabulary, lookahead (uniform or ragged),
element type, temperature per batch or per sequence, row pitch and row offset -- through whichever
kernel set the library picks for each (and each set forced in turn), against the fp64 oracle."""
import numpy as np
import pytest

from gpu_utils import DeviceBatch, assert_parity
from helpers import Case
from paper_2411_00853_b200 import binding
from paper_2411_00853_b200 import workloads as W

pytestmark = [pytest.mark.gpu, pytest.mark.usefixtures("kernel_path")]


def _random_case(seed: int):
    g = np.random.default_rng(1000 + seed)
    cfg = int(g.choice([1, 2, 5]))                                  # fp32 / bf16 fixed lookahead, bf16 ragged
    dtype = str(g.choice(["f32", "bf16", "f16"]))
    B = int(g.choice([1, 2, 3, 7, 16, 18, 19, 33, 70, 150]))
    V = int(g.choice([8, 24, 250, 256, 1000, 1024, 4096, 5000, 12345, 32000, 50264]))
    K = int(g.integers(0, 9)) if cfg != 5 else None
    w = W.make_config(cfg, B=B, V=V, K=K, dtype=dtype)
    T = w.temperature
    if g.random() < 0.5:                                            # a temperature per sequence
        T = g.uniform(0.3, 1.5, size=w.B).astype(np.float32)
    c = Case(w.target_logits, w.draft_logits, w.draft_tokens, w.k_per_row, T, w.uniforms, dtype=w.dtype)
    ld_pad = int(g.choice([0, 0, 8, 3]))
    elem_offset = int(g.choice([0, 0, 0, 8, 1]))
    uniform = cfg != 5 and g.random() < 0.5
    return c, ld_pad, elem_offset, (K if uniform else None)


@pytest.mark.parametrize("seed", range(60))
def test_random_shape(kernel_path, seed):
    c, ld_pad, elem_offset, k_uniform = _random_case(seed)
    dev = DeviceBatch(c, ld_pad=ld_pad, elem_offset=elem_offset)
    got = dev.run(use_k_per_row=k_uniform is None, k_uniform=k_uniform)
    assert binding.last_path() in (binding.PATH_STREAMING, binding.PATH_RING, binding.PATH_CLUSTER)
    assert_parity(c, got, max_excused_frac=0.25 if c.B < 8 else 0.05)
