"""The seeded generators: determinism, dtype-representable values, valid kept sets."""
import numpy as np
import pytest

from paper_2609_39329_b200 import inputs as gen


def small(rule="window_topk", **kw):
    d = dict(d=64, Hq=4, Hkv=2, hd=16, F=64, L=300, N=20, window=8, budget=30, n_obs=4, kept_rule=rule)
    d.update(kw)
    return gen.scaled_config(gen.benchmark_config(2), **d)


def test_benchmark_configs_have_the_stated_shapes():
    c = [gen.benchmark_config(i) for i in range(1, 6)]
    assert [(x.d, x.Hq, x.Hkv, x.hd, x.L, x.N, x.n_layers) for x in c] == [
        (256, 4, 2, 64, 1024, 64, 1), (4096, 32, 8, 128, 32768, 512, 1),
        (4096, 32, 8, 128, 131072, 1024, 32), (3584, 28, 4, 128, 170000, 2048, 28),
        (5120, 32, 8, 128, 65536, 4096, 40)]
    assert all(x.F == x.d for x in c)
    assert [x.budget for x in c] == [128, 3276, 3932, 1700, 2048]
    assert c[3].lam_sweep == (1e-3, 1e-1, 10.0) and c[0].dtype == "fp32"


def test_generation_is_deterministic_and_bf16_representable():
    cfg = small()
    a, b = gen.gen_layer(cfg, 3), gen.gen_layer(cfg, 3)
    for k in a["weights"]:
        np.testing.assert_array_equal(a["weights"][k], b["weights"][k])
    np.testing.assert_array_equal(a["K"], b["K"])
    assert not np.array_equal(a["K"], gen.gen_layer(cfg, 4)["K"])
    for t in (a["K"], a["V"], a["weights"]["Wdown"]):
        np.testing.assert_array_equal(t, gen.round_to_bf16(t))
    assert abs(a["weights"]["Wq"].std() - 0.02) < 2e-3
    # four outlier channels, ten times the spread of the others
    sd = a["K"].reshape(-1, cfg.hd).std(axis=0)
    assert np.sum(sd > 5) == 4 and np.sum((sd > 0.8) & (sd < 1.2)) == cfg.hd - 4


@pytest.mark.parametrize("rule", ["window_topk", "random", "window"])
def test_kept_sets_are_ascending_unique_in_range(rule):
    cfg = small(rule)
    lay = gen.gen_layer(cfg, 0)
    for idx in lay["kept"]:
        assert idx.dtype == np.int32 and len(idx) == cfg.budget
        assert np.all(np.diff(idx) > 0) and idx[0] >= 0 and idx[-1] < cfg.L
    if rule == "window":
        np.testing.assert_array_equal(lay["kept"][0], np.arange(cfg.L - cfg.budget, cfg.L))
    if rule == "window_topk":
        assert np.all(np.isin(np.arange(cfg.L - cfg.window, cfg.L), lay["kept"][1]))
    off, flat = gen.kept_to_csr(lay["kept"])
    assert off.tolist() == [0, cfg.budget, 2 * cfg.budget] and len(flat) == 2 * cfg.budget


def test_topk_ties_go_to_lower_index():
    s = np.array([1.0, 3.0, 3.0, 0.5, 3.0])
    assert gen._topk_lower_index_wins(s, 2).tolist() == [1, 2]


def test_bf16_bits_roundtrip():
    a = gen.round_to_bf16(np.random.default_rng(0).standard_normal(100).astype(np.float32))
    back = (gen.bf16_bits(a).astype(np.uint32) << 16).view(np.float32)
    np.testing.assert_array_equal(a, back)
