"""GPU parity of the float steps between layers and of the two end-to-end networks (reduced
sizes the CPU checker finishes in seconds), through the C ABI.  Every step is a single-rounded
fp32 operation or an exact integer contraction on both sides, so equality is asserted; the stated
bar (<= 1e-5 relative on float outputs) is asserted as well."""
import numpy as np
import pytest
import torch

import paper_1901_09504_b200 as ocs
from ocs_inputs import configs, prng
from oracle import oracle as orc
from paper_1901_09504_b200 import nets

from oracle import net_oracle
from gpu_util import dev, host

pytestmark = pytest.mark.gpu


def test_elementwise_and_pooling_steps():
    x = prng.normal(21, 0, (3, 13, 10, 37), std=2.0)
    b = prng.normal(21, 1, (3, 13, 10, 37), std=2.0)
    x.reshape(-1)[::97] = 0.0
    np.testing.assert_array_equal(host(ocs.ocs_add_relu(dev(x), None, True)), orc.relu(x))
    np.testing.assert_array_equal(host(ocs.ocs_add_relu(dev(x), dev(b), True)), orc.add_relu(x, b, True))
    np.testing.assert_array_equal(host(ocs.ocs_add_relu(dev(x), dev(b), False)), orc.add_relu(x, b, False))
    odd = x.reshape(-1)[:4099].copy()                                        # ragged tail of the vector path
    np.testing.assert_array_equal(host(ocs.ocs_add_relu(dev(odd), None, True)), orc.relu(odd))
    np.testing.assert_array_equal(host(ocs.ocs_maxpool3x3s2(dev(x))), orc.maxpool3x3s2(x))
    x4 = prng.normal(21, 4, (2, 11, 14, 24), std=2.0)                       # C % 4 == 0: the 128-bit form
    np.testing.assert_array_equal(host(ocs.ocs_maxpool3x3s2(dev(x4))), orc.maxpool3x3s2(x4))
    np.testing.assert_array_equal(host(ocs.ocs_global_avgpool(dev(x))), orc.global_avgpool(x))
    nchw = prng.normal(21, 2, (2, 5, 9, 11))
    np.testing.assert_array_equal(host(ocs.ocs_nchw_to_nhwc(dev(nchw))), orc.nchw_to_nhwc(nchw))
    img = prng.normal(21, 5, (2, 3, 20, 30))                                # few channels, several CTAs per image
    np.testing.assert_array_equal(host(ocs.ocs_nchw_to_nhwc(dev(img))), orc.nchw_to_nhwc(img))
    big = prng.normal(21, 3, (2, 70, 33, 35))
    np.testing.assert_array_equal(host(ocs.ocs_nchw_to_nhwc(dev(big))), orc.nchw_to_nhwc(big))


def test_embedding_and_lstm_cell():
    table = prng.uniform(22, 0, (50, 33), -1, 1)
    ids = configs.random_codes(22, 1, (7, 3), 0, 49, np.int32)
    np.testing.assert_array_equal(host(ocs.ocs_embedding(dev(table), dev(ids))), table[ids])
    st = ocs.new_status()
    ids[2, 1] = 50
    ocs.ocs_embedding(dev(table), dev(ids), dev_status=st)
    assert ocs.ocs_poll_status(st) & ocs.DEV_BAD_INDEX
    batch, hidden = 5, 67
    # gate pre-activations over the whole range the routines clamp and mirror on
    g1 = prng.normal(22, 2, (batch, 4 * hidden), std=6.0)
    g2 = prng.normal(22, 3, (batch, 4 * hidden), std=6.0)
    g1[0, :8] = [0.0, -0.0, 100.0, -100.0, 88.0, -88.0, 1e-30, -1e-30]
    g2[0, :8] = 0.0
    c0 = prng.normal(22, 4, (batch, hidden))
    co, ho = orc.lstm_cell(g1, g2, c0)
    cd = dev(c0)
    _, hd = ocs.ocs_lstm_cell(dev(g1), dev(g2), cd)
    np.testing.assert_array_equal(host(cd).view(np.uint32), co.view(np.uint32))
    np.testing.assert_array_equal(host(hd).view(np.uint32), ho.view(np.uint32))


def test_resnet50_stack_reduced_end_to_end():
    """The full ResNet-50 conv/fc stack (r = 0.01, 8-bit weights and activations) on 2 images of 64x64."""
    cfg = configs.config4(batch=2, image=64)
    ref_logits, ref = net_oracle.resnet50(cfg)
    st = ocs.new_status()
    layers = nets.prepare_resnet50(cfg, torch.device("cuda"), dev_status=st)
    logits, t = nets.resnet50_forward(cfg, layers, dev(cfg["X"]), keep=True, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    for name in ["conv1", "pool"] + [s.name for s in cfg["layers"][1:]] + ["avgpool", "fc"]:
        np.testing.assert_allclose(host(t[name]), ref[name], rtol=1e-5, atol=0, err_msg=name)
        np.testing.assert_array_equal(host(t[name]), ref[name], err_msg=name)
    np.testing.assert_array_equal(host(logits), ref_logits)
    assert np.isfinite(ref_logits).all() and np.abs(ref_logits).max() > 0


def test_lstm_language_model_reduced_end_to_end():
    """Two-layer LSTM, hidden 650, r = 0.02, 6-bit weights, 8-bit signed activations; vocabulary 3000,
    batch 4, 6 time steps."""
    cfg = configs.config5(vocab=3000, batch=4, seq=6)
    ref_logits, ref = net_oracle.lstm(cfg)
    st = ocs.new_status()
    layers = nets.prepare_lstm(cfg, torch.device("cuda"), dev_status=st)
    logits, t = nets.lstm_forward(cfg, layers, dev(cfg["tokens"]), keep=True, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(t["emb"]), ref["emb"])
    np.testing.assert_array_equal(host(t["tops"]), ref["tops"])
    for l in range(2):
        np.testing.assert_array_equal(host(t["c"][l]), ref["c"][l])
    np.testing.assert_allclose(host(logits), ref_logits, rtol=1e-5, atol=0)
    np.testing.assert_array_equal(host(logits), ref_logits)


def test_lstm_with_folded_duplicates_gives_the_same_logits():
    """6-bit codes: the copies folded back into their source channels, no gather in any GEMM, same outputs."""
    cfg = configs.config5(vocab=3000, batch=4, seq=6)
    ref_logits, ref = net_oracle.lstm(cfg)
    st = ocs.new_status()
    layers = nets.prepare_lstm(cfg, torch.device("cuda"), dev_status=st, fold=True)
    assert all(L.S == 0 for name, L in layers.items() if name != "emb")
    logits, t = nets.lstm_forward(cfg, layers, dev(cfg["tokens"]), keep=True, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(t["tops"]), ref["tops"])
    np.testing.assert_array_equal(host(logits), ref_logits)


def test_batched_preparation_equals_per_layer_calls():
    """ocs_split_quantize_batch on a mix of layer shapes (short rows, long rows, 1x1 and 3x3, fully connected, S = 0)
    gives every layer the bytes of its own ocs_split_quantize call, which in turn equal the checker's."""
    shapes = [(64, 64, 1, 1), (64, 64, 3, 3), (256, 64, 1, 1), (128, 128, 3, 3), (512, 256, 1, 1), (128, 1024, 1, 1),
              (96, 512, 3, 3), (1000, 2048), (33, 20), (16, 8)]
    Ws = []
    for i, sh in enumerate(shapes):
        W = prng.laplace(61, i, sh, 0.02)
        W.reshape(-1)[prng.distinct_positions(61, 100 + i, W.size, 4)] *= 20
        Ws.append(W)
    Ss = [ocs.ocs_num_splits(W.shape[1], 0.02) for W in Ws]
    Ss[-1] = 0
    st = ocs.new_status()
    outs = ocs.ocs_split_quantize_batch([dev(W) for W in Ws], Ss, 8, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    for W, S, (codes, scale, idx_map) in zip(Ws, Ss, outs):
        c1, s1, _, i1, _, _ = ocs.ocs_split_quantize(dev(W), S, 8, ocs.CLIP_NONE, dev_status=st)
        cols = (W.shape[1] + S) * int(np.prod(W.shape[2:]))
        np.testing.assert_array_equal(host(idx_map), host(i1))
        assert host(scale)[0] == host(s1)[0]
        np.testing.assert_array_equal(host(codes)[:, :cols], host(c1)[:, :cols])
        Wp, idx_o, _, _ = orc.split(W, S, 0.0)
        wc, wscale = orc.quantize(Wp, 8, True, orc.maxabs(Wp))
        np.testing.assert_array_equal(host(idx_map), idx_o)
        assert host(scale)[0] == np.float32(wscale)
        np.testing.assert_array_equal(host(codes)[:, :cols], wc.reshape(W.shape[0], -1))
    assert ocs.ocs_poll_status(st) == 0
    with pytest.raises(ocs.OcsError) as e:                       # 3 x 49 weights per filter: not a multiple of 4
        ocs.ocs_split_quantize_batch([dev(prng.laplace(61, 50, (8, 3, 7, 7), 0.1))], [1], 8)
    assert e.value.status == 4
