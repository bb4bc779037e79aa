"""GPU parity at the benchmark's full sizes, in the launch configuration the benchmark times
(trdq_run_layers over a layer list): activation codes are compared in full, GEMM outputs on sampled rows
(first and last tile plus a seeded sample) that the CPU oracle can compute one by one."""
import numpy as np
import pytest

from oracle import trdq_oracle as O
from paper_2503_06564_b200 import workloads as WL
from tests.util import bf16_to_f32_np, check_output, to_dev_bf16

pytestmark = pytest.mark.gpu


def _run_layer(wl, layer_idx, t, sample=384):
    import torch
    from paper_2503_06564_b200 import trdq
    inp = WL.make_layer_inputs(wl, layer_idx)
    K, N, M = inp.layer.K, inp.layer.N, inp.M
    rot = trdq.Rotation(K, inp.t_bounds, inp.signs, inp.smooth)
    wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(inp.w), wl.wbits)
    xd, bias_d = to_dev_bf16(inp.x), to_dev_bf16(inp.bias)
    codes = torch.empty((M, K), dtype=torch.int8, device="cuda")
    scales = torch.empty((M,), dtype=torch.float32, device="cuda")
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    layers = trdq.LayerList()
    layers.add(rot, wts, xd, codes, scales, bias_d, y)
    trdq.trdq_run_layers(layers, t)
    torch.cuda.synchronize()

    g = O.group_of(inp.t_bounds, t)
    assert g == rot.group_of(t)
    act, wv = O.fused_vectors(inp.signs[g], None if inp.smooth is None else inp.smooth[g])
    q_ref, sx_ref = O.rotate_quantize(inp.x, act)
    assert np.array_equal(scales.cpu().numpy(), sx_ref)
    assert np.array_equal(codes.cpu().numpy(), q_ref)
    rows = WL.sample_rows(wl, layer_idx, M, sample)
    if wl.wbits == 8:
        qw_ref, sw_ref = O.prepare_w8(inp.w, wv)
        y_ref = O.linear_w8_rows(q_ref, sx_ref, qw_ref, sw_ref, inp.bias, rows)
    else:
        pk_ref, sw4_ref = O.prepare_w4(inp.w, wv)
        y_ref = O.linear_w4_rows(q_ref, sx_ref, pk_ref, sw4_ref, inp.bias, rows)
    y_rows = bf16_to_f32_np(y[torch.from_numpy(rows).cuda()])
    l2, ulps = check_output(y_rows, y_ref, max_ulp=2.0, rel_l2=2e-3)
    assert ulps <= 1.0
    assert trdq.trdq_device_status() == 0


@pytest.mark.parametrize("layer_idx", [0, 1, 2, 3])
def test_dit_xl2_256px_all_layers(layer_idx):
    """Configuration the headline metric is quoted on: M = 4096, every layer shape, a time-step of the last group."""
    _run_layer(WL.WORKLOADS[1], layer_idx, t=980)


@pytest.mark.parametrize("layer_idx", [0, 1, 2, 3])
def test_dit_xl2_512px_all_layers(layer_idx):
    """M = 16384, every layer shape (K = 1152 rows and the K = 4608 rows of fc2), one time-step per group across the layers."""
    _run_layer(WL.WORKLOADS[2], layer_idx, t=(400, 0, 999, 600)[layer_idx], sample=256)


@pytest.mark.parametrize("layer_idx", [0, 1, 2, 3, 4, 5])
def test_pixart_1024px_all_layers_and_cross_attention(layer_idx):
    """M = 32768 on the four block linears; the cross-attention K and V projections on their 960 text rows (all rows)."""
    wl = WL.WORKLOADS[3]
    _run_layer(wl, layer_idx, t=(10, 260, 510, 999, 740, 250)[layer_idx], sample=960 if layer_idx >= 4 else 256)


@pytest.mark.parametrize("layer_idx", [0, 1, 2, 3])
def test_video_dit_w4a8_all_layers(layer_idx):
    """M = 16384, int4 weights; fc2 has 36 scale groups along K."""
    _run_layer(WL.WORKLOADS[4], layer_idx, t=(700, 0, 350, 999)[layer_idx], sample=256)


def test_run_layers_follows_the_time_step_schedule():
    """A list of layers over a few sampling steps: every step picks its group (switches included) and the result
    equals the individual calls; inconsistent lists are refused before anything is launched."""
    import torch
    from paper_2503_06564_b200 import trdq
    wl = WL.WORKLOADS[1]
    layers = trdq.LayerList()
    singles = []
    for li in (1, 3):
        inp = WL.make_layer_inputs(wl, li, M=200)
        rot = trdq.Rotation(inp.layer.K, inp.t_bounds, inp.signs, inp.smooth)
        wts = trdq.trdq_prepare_weights(rot, to_dev_bf16(inp.w), 8)
        xd, bias_d = to_dev_bf16(inp.x), to_dev_bf16(inp.bias)
        codes = torch.empty((200, inp.layer.K), dtype=torch.int8, device="cuda")
        scales = torch.empty((200,), dtype=torch.float32, device="cuda")
        y = torch.empty((200, inp.layer.N), dtype=torch.bfloat16, device="cuda")
        layers.add(rot, wts, xd, codes, scales, bias_d, y)
        singles.append((rot, wts, xd, bias_d, y))
    ts = wl.timesteps()
    seen_groups = set()
    for t in (int(ts[0]), int(ts[9]), int(ts[10]), int(ts[49])):      # steps 9 -> 10 cross a group boundary
        trdq.trdq_run_layers(layers, t)
        for rot, wts, xd, bias_d, y in singles:
            c, s = trdq.trdq_rotate_quantize(rot, t, xd)
            assert torch.equal(trdq.trdq_linear(wts, t, c, s, bias_d), y)
            seen_groups.add(rot.group_of(t))
    assert seen_groups == {4, 3, 0}
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_run_layers(layers, 1000)
    assert e.value.status == 4
    # a layer whose rotation and weights were built for different K
    bad = trdq.LayerList()
    rot_a, wts_a, xd_a, bias_a, y_a = singles[0]
    rot_b = singles[1][0]
    bad.add(rot_b, wts_a, xd_a, torch.empty((200, rot_b.K), dtype=torch.int8, device="cuda"),
            torch.empty((200,), dtype=torch.float32, device="cuda"), bias_a, y_a)
    with pytest.raises(trdq.TrdqError) as e:
        trdq.trdq_run_layers(bad, 0)
    assert e.value.status == 10


def test_run_layers_block_with_shared_attention_and_fused_gelu():
    """One transformer block's four linears as a layer list in which the attention linears see the conditional rows
    only (the unconditional branch reuses the conditional attention, Sec. 3.3) and the first MLP linear carries its GELU
    in the epilogue.  Every op must equal the stand-alone calls bit for bit, and the oracle on sampled rows."""
    import torch
    from paper_2503_06564_b200 import trdq
    rng = np.random.default_rng(123)
    hidden, M, M_cond = 1152, 1024, 512
    bounds = WL.group_bounds(2)
    shapes = [(hidden, 3 * hidden, M_cond, 0), (hidden, hidden, M_cond, 0), (hidden, 4 * hidden, M, 1), (4 * hidden, hidden, M, 0)]
    layers = trdq.LayerList()
    keep = []
    for K, N, rows, act in shapes:
        signs = (rng.integers(0, 2, (2, K)) * 2 - 1).astype(np.int8)
        rot = trdq.Rotation(K, bounds, signs)
        w_bits = WL.to_bf16_bits(rng.standard_normal((N, K)) * 0.05)
        bias_bits = WL.to_bf16_bits(rng.standard_normal(N) * 0.1)
        w = trdq.trdq_prepare_weights(rot, to_dev_bf16(w_bits), 8)
        x_bits = WL.to_bf16_bits(rng.standard_normal((rows, K)))
        x, bias = to_dev_bf16(x_bits), to_dev_bf16(bias_bits)
        codes = torch.empty((rows, K), dtype=torch.int8, device="cuda")
        scales = torch.empty((rows,), dtype=torch.float32, device="cuda")
        y = torch.empty((rows, N), dtype=torch.bfloat16, device="cuda")
        layers.add(rot, w, x, codes, scales, bias, y, act=act)
        keep.append((rot, w, x, x_bits, bias, bias_bits, signs, codes, scales, y, act))
    t = 700
    trdq.trdq_run_layers(layers, t)
    g = 1
    for rot, w, x, x_bits, bias, bias_bits, signs, codes, scales, y, act in keep:
        c2, s2 = trdq.trdq_rotate_quantize(rot, t, x)
        y2 = trdq.trdq_linear_act(w, t, c2, s2, bias, act=act)
        assert torch.equal(c2, codes) and torch.equal(s2, scales) and torch.equal(y2, y)
        a, _ = O.fused_vectors(signs[g], None)
        c_ref, s_ref = O.rotate_quantize(x_bits, a)
        assert np.array_equal(codes.cpu().numpy(), c_ref) and np.array_equal(scales.cpu().numpy(), s_ref)
        wq, sw = w.view_tensors(g)
        rows = np.arange(0, x.shape[0], 37, dtype=np.int64)
        y_ref = O.linear_w8_rows(c_ref, s_ref, wq.cpu().numpy(), sw.cpu().numpy(), bias_bits, rows, act=act)
        check_output(bf16_to_f32_np(y)[rows], y_ref, tiny=2.0 ** -100 if act else 0.0)
    assert trdq.trdq_device_status() == 0
