"""The seeded workload generator: reproducible bits, recipe facts that the other tests rely on."""
import numpy as np

from paper_2308_10037_b200 import datagen


def test_bits_do_not_depend_on_the_thread_count():
    wl = datagen.scaled(datagen.WORKLOADS["cfg5"], 3 * datagen.CHUNK_ROWS + 17)
    X1, y1, w1, b1 = datagen.generate(wl, threads=1)
    X4, y4, w4, b4 = datagen.generate(wl, threads=4)
    assert np.array_equal(X1, X4) and np.array_equal(y1, y4) and np.array_equal(w1, w4) and b1 == b4
    # a shorter instance of the same recipe is a prefix of the longer one (chunk-keyed streams)
    Xs, ys, _, _ = datagen.generate(datagen.scaled(datagen.WORKLOADS["cfg5"], datagen.CHUNK_ROWS), threads=2)
    assert np.array_equal(Xs, X1[:datagen.CHUNK_ROWS])


def test_recipes():
    # cfg2: per-feature scales in [0.5, 2]; labels balanced for b* = 0
    X, y, w, b = datagen.generate(datagen.scaled(datagen.WORKLOADS["cfg2"], 50_000), threads=2)
    sd = X.std(axis=0)
    assert X.dtype == np.float32 and y.dtype == np.float32 and set(np.unique(y)) <= {0.0, 1.0}
    assert 0.45 < sd.min() and sd.max() < 2.1 and b == 0.0 and abs(y.mean() - 0.5) < 0.02
    # cfg3: 26 of 256 planted weights are non-zero
    assert np.count_nonzero(datagen.planted_w(datagen.WORKLOADS["cfg3"])) == 26
    # cfg4: features in [0, 1), about half the labels positive
    X, y, w, b = datagen.generate(datagen.scaled(datagen.WORKLOADS["cfg4"], 4_000), threads=2)
    assert X.min() >= 0.0 and X.max() < 1.0 and abs(y.mean() - 0.5) < 0.05
    # cfg5: the last 19 of 64 columns are 0/1 with rate ~0.1; about 1 % positives
    X, y, w, b = datagen.generate(datagen.scaled(datagen.WORKLOADS["cfg5"], 200_000), threads=2)
    tail = X[:, 64 - 19:]
    assert set(np.unique(tail)) <= {0.0, 1.0} and abs(tail.mean() - 0.1) < 0.01
    assert len(np.unique(X[:, 0])) > 1000 and 0.005 < y.mean() < 0.02
    # the x_out path writes into the caller's buffer
    buf = np.empty((1000, 32), dtype=np.float32)
    Xo, _, _, _ = datagen.generate(datagen.scaled(datagen.WORKLOADS["cfg1"], 1000), threads=1, x_out=buf)
    assert Xo is buf
