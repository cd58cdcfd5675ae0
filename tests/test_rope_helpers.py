"""Host helpers that build the rotation tables: Eq. 8 indices against the oracle's statement of Eq. 8 and hand values,
table shapes and the plane-rotation property through the oracle's rotate_pairs."""
import numpy as np

from oracle import hybrid_attention as oa
from paper_2604_10103_b200 import rope


def test_relative_temporal_indices_match_eq8():
    for i in (3, 4, 20, 21, 22, 100, 601):
        assert rope.relative_temporal_indices(i, 21) == oa.relative_temporal_indices(i, 21)
    assert rope.relative_temporal_indices(6, 21) == [4, 5, 6]
    assert rope.relative_temporal_indices(600, 21) == [19, 20, 21]
    assert rope.relative_temporal_indices(5, 21, chunk_frames=1) == [5]


def test_angle_tables_shape_and_rotation():
    pos = rope.chunk_positions(last_frame=30, t0=21, chunk_frames=3, height=2, width=3)
    assert pos.shape == (18, 3) and pos[:, 0].min() == 19 and pos[:, 0].max() == 21
    assert (pos[:6, 0] == 19).all() and pos[5].tolist() == [19, 1, 2]
    cos, sin = rope.angle_tables(pos, (2, 1, 1))
    assert cos.shape == sin.shape == (18, 4) and cos.dtype == np.float32
    assert np.allclose(cos ** 2 + sin ** 2, 1.0, atol=1e-6)
    # first pair of an axis turns by exactly the position (frequency 1): token 5 -> t = 19
    assert np.isclose(cos[5, 0], np.cos(19.0), atol=1e-6) and np.isclose(sin[5, 3], np.sin(2.0), atol=1e-6)
    x = np.random.default_rng(0).standard_normal((18, 8))
    y = oa.rotate_pairs(x, cos, sin)
    assert np.allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1), rtol=1e-6)
