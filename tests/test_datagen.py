"""The seeded input generator: its native filler for large tensors draws the same values as the
numpy formulation, and the realised zero density matches the request."""
import numpy as np

import datagen


def test_native_filler_equals_numpy_formulation():
    for seed, (M, K), z in ((3, (512, 384), 0.42), (20260916, (300, 1024), 0.3288), (7, (256, 512), 0.0)):
        a = datagen.trits(seed, M, K, z)
        b = datagen.trits(seed, M, K, z, native=False)
        assert a.dtype == np.int8 and np.array_equal(a, b)
        assert abs((a == 0).mean() - z) < 0.01
        assert abs((a == 1).mean() - (a == -1).mean()) < 0.01


def test_any_element_can_be_drawn_on_its_own():
    u = datagen.uniform(11, datagen.STREAM_X, 0, 1000)
    assert np.array_equal(u[123:130], datagen.uniform(11, datagen.STREAM_X, 123, 7))
