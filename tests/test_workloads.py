"""The synthetic input recipes: shapes, determinism and value structure."""
import numpy as np

from paper_2503_06564_b200 import workloads as WL


def test_bf16_round_trip_and_ties():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0, 3.0e38], np.float32)
    bits = WL.f32_to_bf16_bits(x)
    back = WL.bf16_bits_to_f32(bits)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == np.float32(1.015625)
    assert back[3] == -2.5 and back[4] == 0.0
    assert np.array_equal(WL.f32_to_bf16_bits(back), bits)


def test_workload_shapes_match_configs():
    w = WL.WORKLOADS
    assert [x.M for x in w] == [256, 4096, 16384, 32768, 16384]
    assert [x.num_groups for x in w] == [2, 5, 5, 4, 3]
    assert [x.steps for x in w][1:] == [50, 50, 20, 30]
    assert w[4].wbits == 4 and all(x.wbits == 8 for x in w[:4])
    for wl in w:
        for layer in wl.layers + wl.extra_layers:
            assert layer.K % WL.BLOCK == 0 and layer.N % 16 == 0
    assert [(l.K, l.N) for l in w[1].layers] == [(1152, 3456), (1152, 1152), (1152, 4608), (4608, 1152)]
    assert [(l.K, l.N, l.M) for l in w[3].extra_layers] == [(4096, 1152, 960)] * 2


def test_timesteps_and_bounds():
    assert WL.group_bounds(2).tolist() == [0, 500, 1000]
    assert WL.group_bounds(3).tolist() == [0, 333, 666, 1000]
    ts = WL.sampling_timesteps(50)
    assert ts[0] == 980 and ts[-1] == 0 and np.all(np.diff(ts) < 0)
    for wl in WL.WORKLOADS[1:]:
        b = wl.t_bounds
        g = np.searchsorted(b, wl.timesteps(), side="right") - 1
        assert set(g.tolist()) == set(range(wl.num_groups))
        assert int((np.diff(g) != 0).sum()) == wl.num_groups - 1     # G-1 switches per run


def test_inputs_are_seeded_and_structured():
    wl = WL.WORKLOADS[0]
    a = WL.make_layer_inputs(wl, 0, M=16)
    b = WL.make_layer_inputs(wl, 0, M=16)
    assert np.array_equal(a.x, b.x) and np.array_equal(a.w, b.w) and np.array_equal(a.signs, b.signs)
    assert a.x.dtype == np.uint16 and a.x.shape == (16, 1024) and a.w.shape == (1024, 1024)
    assert set(np.unique(a.signs).tolist()) == {-1, 1} and a.signs.shape == (2, 1024)
    assert not np.array_equal(a.signs[0], a.signs[1])
    ch = WL.outlier_channels(wl, 0, 1024)
    assert ch.tolist() == [(131 * i + 7) % 1024 for i in range(8)]
    assert len(set((ch // 128).tolist())) == 8          # one per 128-block
    x = WL.bf16_bits_to_f32(a.x)
    others = np.setdiff1d(np.arange(1024), ch)
    assert np.abs(x[:, ch]).mean() > 20 * np.abs(x[:, others]).mean()
    assert a.smooth is None
    wl1 = WL.WORKLOADS[1]
    c = WL.make_layer_inputs(wl1, 1, M=32)
    assert c.smooth.shape == (5, 1152) and np.all(c.smooth > 0)
    assert WL.outlier_channels(wl1, 1, 1152).size == 12 and WL.outlier_channels(wl1, 3, 4608).size == 47


def test_sample_rows_cover_edges():
    wl = WL.WORKLOADS[2]
    rows = WL.sample_rows(wl, 0, 16384, 2048)
    assert rows[0] == 0 and rows[-1] == 16383 and rows.size >= 2048
    assert np.all(np.isin(np.arange(128), rows)) and np.all(np.isin(np.arange(16384 - 128, 16384), rows))
