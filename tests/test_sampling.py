"""The samplers of the full-size parity tests (no GPU): every row tile of the token axis and every
weight-gradient output tile must hold a sample, and a ragged tail is taken whole."""
import numpy as np

from tests.helpers import DW_TILE, ROW_TILE, stratified_entries, stratified_tokens


def test_sampling_covers_every_tile():
    # the sampler itself (no GPU work): every row tile and every weight-gradient tile holds a sample
    rng = np.random.default_rng(0)
    for T in (16384, 16384 + 77, 200):
        tok = stratified_tokens(T, rng)
        assert set(range(-(-T // ROW_TILE))) == set(int(r) // ROW_TILE for r in tok)
        assert all(r in tok for r in range(T - T % ROW_TILE, T))
    m_, l_, k_ = stratified_entries(8, 4096, 1376, rng)
    assert len(m_) >= 4096
    tiles = set(zip(m_.tolist(), (l_ // DW_TILE[0]).tolist(), (k_ // DW_TILE[1]).tolist()))
    assert len(tiles) == 8 * 32 * 6
