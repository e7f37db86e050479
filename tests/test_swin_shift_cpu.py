"""Host-side pieces of the shifted-window blocks: row permutations and masks, checked against a plain roll of the
token grid (the definition), without reference to the index formulas of the generator."""
import numpy as np

from ivit_inputs.gen import SHIFT_MASK, shift_indices, shift_mask


def _window_major_to_grid(X, B, res, window):
    """[B*res*res, C] rows in window-major order -> [B, res, res, C]."""
    w = res // window
    C = X.shape[1]
    return X.reshape(B, w, w, window, window, C).transpose(0, 1, 3, 2, 4, 5).reshape(B, res, res, C)


def _grid_to_window_major(G, window):
    B, res, _, C = G.shape
    w = res // window
    return G.reshape(B, w, window, w, window, C).transpose(0, 1, 3, 2, 4, 5).reshape(B * res * res, C)


def test_shift_index_is_a_roll_of_the_token_grid():
    B, res, window = 2, 14, 7
    rng = np.random.default_rng(0)
    X = rng.integers(-128, 128, (B * res * res, 5)).astype(np.int8)
    fwd, inv = shift_indices(B, res, window)
    grid = _window_major_to_grid(X, B, res, window)
    rolled = np.roll(grid, shift=(-(window // 2), -(window // 2)), axis=(1, 2))
    np.testing.assert_array_equal(X[fwd], _grid_to_window_major(rolled, window))
    np.testing.assert_array_equal(X[fwd][inv], X)
    assert sorted(fwd.tolist()) == list(range(B * res * res))


def test_shift_mask_separates_the_wrapped_regions():
    res, window = 28, 7
    s = window // 2
    m = shift_mask(res, window)
    w = res // window
    assert m.shape == (w * w, window * window, window * window)
    # label every token of the rolled grid by the image side it came from: rows/columns that wrapped around
    # (the last s of the rolled grid) may not attend to the rest of their window
    yy, xx = np.meshgrid(np.arange(res), np.arange(res), indexing="ij")
    wrapped_y, wrapped_x = yy >= res - s, xx >= res - s
    for wy in range(w):
        for wx in range(w):
            sl = (slice(wy * window, (wy + 1) * window), slice(wx * window, (wx + 1) * window))
            a, b = wrapped_y[sl].reshape(-1), wrapped_x[sl].reshape(-1)
            same = (a[:, None] == a[None, :]) & (b[:, None] == b[None, :])
            np.testing.assert_array_equal(m[wy * w + wx] == 0, same)
    assert set(np.unique(m).tolist()) == {0, SHIFT_MASK}
    # interior windows are unmasked; the last window has four regions
    assert not m[0].any() and len(np.unique((m[-1] == 0).sum(1))) == 3
