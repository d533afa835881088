"""Pins of the oracle's frame pre-processing (Section 5.1: maximum of the two latest raw frames, pixel intensity,
210 x 160 -> 84 x 84, four-frame state).  CPU only."""
import numpy as np


def _area_mean_by_upsampling(grey):
    """Independent statement of the area average: repeat every source row twice and every source column 21 times
    (420 x 3360), then every output pixel is the plain mean of a 5 x 40 block; round half up."""
    up = np.repeat(np.repeat(grey.astype(np.int64), 2, axis=0), 21, axis=1)
    assert up.shape == (420, 3360)
    sums = up.reshape(84, 5, 84, 40).sum(axis=(1, 3))
    return ((2 * sums + 200) // 400).astype(np.uint8)


def _grey(rgb):
    r, g, b = (rgb[..., k].astype(np.int64) for k in range(3))
    return ((77 * r + 150 * g + 29 * b + 128) >> 8).astype(np.uint8)


def test_matches_block_means_of_the_upsampled_image(orc):
    rng = np.random.RandomState(0)
    a = rng.randint(0, 256, (3, 210, 160, 3), dtype=np.uint8)
    b = rng.randint(0, 256, (3, 210, 160, 3), dtype=np.uint8)
    prev = rng.randint(0, 256, (3, 84, 84, 4), dtype=np.uint8)
    out = orc.preprocess(a, b, prev)
    for e in range(3):
        want = _area_mean_by_upsampling(_grey(np.maximum(a[e], b[e])))
        assert np.array_equal(out[e, :, :, 3], want)
        assert np.array_equal(out[e, :, :, :3], prev[e, :, :, 1:])          # the three older frames move down
    first = orc.preprocess(a, b, None)
    for k in range(4):
        assert np.array_equal(first[..., k], out[..., 3])                   # after a reset the new frame fills the state


def test_constant_and_pure_colour_images(orc):
    z = np.zeros((1, 210, 160, 3), np.uint8)
    for v in (0, 1, 127, 255):
        assert np.all(orc.preprocess(z, z + v)[..., 3] == v)               # grey levels are kept, white stays 255
    for k, w in enumerate((77, 150, 29)):
        img = z.copy()
        img[..., k] = 200
        assert np.all(orc.preprocess(img, z)[..., 3] == (w * 200 + 128) >> 8)
    # the maximum is per colour channel: red in one frame and green in the other add up in the intensity
    red, green = z.copy(), z.copy()
    red[..., 0], green[..., 1] = 255, 255
    assert np.all(orc.preprocess(red, green)[..., 3] == (77 * 255 + 150 * 255 + 128) >> 8)


def test_hand_computed_rows_and_columns(orc):
    z = np.zeros((1, 210, 160, 3), np.uint8)
    # intensity = source row index: output row 0 averages rows 0, 1, 2 with weights 2, 2, 1 -> 0.8 -> 1;
    # output row 1 averages rows 2, 3, 4 with weights 1, 2, 2 -> 3.2 -> 3; output row 2 is rows 5, 6, 7 -> 5.8 -> 6
    img = z.copy()
    img[0] += np.arange(210, dtype=np.uint8)[:, None, None]
    out = orc.preprocess(img, z)[0, :, :, 3]
    assert out[0, 0] == 1 and out[1, 0] == 3 and out[2, 0] == 6 and np.all(out == out[:, :1])
    # intensity = source column index: output column 0 covers [0, 40/21): columns 0 (21 parts) and 1 (19 parts)
    # -> 19/40 -> 0; output column 1 covers [40/21, 80/21): column 1 (2 parts), 2 (21), 3 (17) -> 95/40 = 2.375 -> 2
    img = z.copy()
    img[0] += np.arange(160, dtype=np.uint8)[None, :, None]
    out = orc.preprocess(img, z)[0, :, :, 3]
    assert out[0, 0] == 0 and out[0, 1] == 2 and np.all(out == out[:1, :])
    # a single bright source pixel spreads over the output pixels it overlaps, in proportion to the shared area:
    # source (2, 1) lies half in output row 0 and half in row 1, and 19/21 in output column 0, 2/21 in column 1
    img = z.copy()
    img[0, 2, 1] = 255
    out = orc.preprocess(img, z)[0, :, :, 3].astype(int)
    full = 255 * 42 * 84                      # weight 42 x 84 (in 1/84 units) is half a row times a whole column
    assert out[0, 0] == (full * 19 // 21 + 16800) // 33600 and out[1, 0] == out[0, 0]
    assert out[0, 1] == (full * 2 // 21 + 16800) // 33600 and out[2:, :].sum() == 0 and out[:, 2:].sum() == 0


def test_stack_push_is_the_stacking_half_of_the_preprocessing(orc):
    """The frame stack by itself: it must give what the whole pre-processing gives when the newest frame is the
    pre-processed one; four pushes of known planes leave them in order, oldest first; a restart fills the state."""
    rng = np.random.RandomState(4)
    a = rng.randint(0, 256, (3, 210, 160, 3), dtype=np.uint8)
    b = rng.randint(0, 256, (3, 210, 160, 3), dtype=np.uint8)
    prev = rng.randint(0, 256, (3, 84, 84, 4), dtype=np.uint8)
    whole = orc.preprocess(a, b, prev)
    assert np.array_equal(orc.stack_push(prev, whole[..., 3]), whole)
    assert np.array_equal(orc.stack_push(prev, whole[..., 3], np.ones(3, np.uint8)), orc.preprocess(a, b, None))
    # planes 1, 2, 3, 4 pushed one after the other into a state of zeros
    st = np.zeros((2, 84, 84, 4), np.uint8)
    for v in (1, 2, 3, 4):
        st = orc.stack_push(st, np.full((2, 84, 84), v, np.uint8))
    assert np.array_equal(st[0, 5, 7], [1, 2, 3, 4]) and np.all(st == np.array([1, 2, 3, 4], np.uint8))
    # a restart in environment 1 only
    st2 = orc.stack_push(st, np.full((2, 84, 84), 9, np.uint8), np.array([0, 1], np.uint8))
    assert np.all(st2[0] == np.array([2, 3, 4, 9], np.uint8)) and np.all(st2[1] == 9)
    # brute force on random data, pixel by pixel
    planes = rng.randint(0, 256, (3, 84, 84), dtype=np.uint8)
    out = orc.stack_push(prev, planes, np.array([0, 1, 0], np.uint8))
    for e, y, x in ((0, 0, 0), (0, 83, 83), (1, 40, 2), (2, 17, 60)):
        want = [planes[e, y, x]] * 4 if e == 1 else list(prev[e, y, x, 1:]) + [planes[e, y, x]]
        assert list(out[e, y, x]) == want
