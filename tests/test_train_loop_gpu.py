"""End-to-end loop (model gradients -> quantize -> server step -> selector) on the GPU."""
import pytest

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("selector", ["window", "sarsa"])
def test_loop_trains_and_reports_the_library_share(selector):
    from paper_1804_08066_b200.train_loop import run
    r = run(iters=40, workers=4, selector=selector, seed=1)
    assert r["parameters"] == 3 * 32 * 9 + 32 + 32 * 64 * 9 + 64 + 64 * 128 * 9 + 128 + 2048 * 256 + 256 + 2560 + 10
    assert all(1 <= b <= 8 for b in r["bits_chosen"])
    if selector == "sarsa":
        assert all(b2 >= b1 for b1, b2 in zip(r["bits_chosen"], r["bits_chosen"][1:]))
        assert min(r["bits_chosen"]) >= 2
    assert r["last_loss"] < r["first_loss"]                  # quantized SGD still learns
    assert 0 < r["libmqgrad_share_pct"] < 100
    assert r["uplink_bytes_per_iter"] < r["uplink_bytes_fp32"]
