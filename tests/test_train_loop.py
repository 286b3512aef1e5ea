"""The training loop's schedule and call plan (no GPU: the step is a recorder)."""
import numpy as np
import pytest

from paper_1606_08495_b200.train import learning_rate, train


def test_linear_schedule_endpoints_and_floor():
    assert learning_rate(0.025, 0, 1000) == pytest.approx(0.025)
    assert learning_rate(0.025, 500, 999) == pytest.approx(0.0125)
    assert learning_rate(0.025, 10**9, 1000) == pytest.approx(0.025 * 1e-4)
    assert learning_rate(0.02, 123, 1000, "epoch", epoch=1, epochs=4) == pytest.approx(0.015)
    with pytest.raises(ValueError):
        learning_rate(0.1, 0, 1, "cosine")


def test_call_plan_with_interleaving():
    chunks = [np.array([1, 2, -1, 3], dtype=np.int32), np.array([4, -1], dtype=np.int32)]
    calls = []
    n = train(lambda t, lr, num, ph, st: calls.append((len(t), round(lr, 6), num, ph, st)), chunks, epochs=2,
              lr0=0.1, stride=3)
    assert n == len(calls) == 2 * 2 * 3
    # every chunk visit: phases 0, 1, 2 with one step number and one learning rate
    for k in range(0, 12, 3):
        trio = calls[k:k + 3]
        assert [c[3] for c in trio] == [0, 1, 2] and len({(c[0], c[1], c[2], c[4]) for c in trio}) == 1
    assert [calls[k][2] for k in range(0, 12, 3)] == [0, 1, 2, 3]
    lrs = [calls[k][1] for k in range(0, 12, 3)]
    assert lrs[0] == pytest.approx(0.1) and all(a > b for a, b in zip(lrs, lrs[1:]))   # 8 words in all
    assert lrs[1] == pytest.approx(0.1 * (1 - 3 / 9.0), abs=1e-6)
