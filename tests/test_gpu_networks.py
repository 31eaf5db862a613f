"""GPU parity on network-shaped workloads: every activation tensor of the CUDA forward pass
against the CPU oracle's forward pass from the same image, bit-exact; logits within 1e-6 relative.

The oracle always starts from the image (nothing it consumes comes from the GPU).  Full-size
networks run on the GPU at the batch size the benchmark uses; the oracle recomputes a few of
the images one by one (images of a batch are independent).
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def psb():
    import paper_1904_02205_b200 as p

    return p


def _run_gpu(psb, layers, net, batch, level_mask, seed, uniform_log2k, fc_log2k=None, kmaps=None):
    import torch
    from paper_1904_02205_b200.network import Network

    ctx = psb.Context(0)
    nw = Network(ctx, layers, net, batch, level_mask, kmaps=kmaps, uniform_log2k=uniform_log2k, fc_log2k=fc_log2k)
    nw.sample(seed)
    logits = nw.forward(torch.from_numpy(net["image"][:batch]).to(ctx.device))
    assert ctx.device_status() == 0
    return ctx, nw, logits.cpu().numpy()


def _compare(nw, logits, oracle, layers, net, images_idx, seed, uniform_log2k, fc_log2k=None, kmaps=None):
    idx = np.asarray(images_idx)
    km = None if kmaps is None else {r: m[idx] for r, m in kmaps.items()}
    acts, ref_logits = oracle.run_network(layers, net, net["image"][idx], seed, uniform_log2k=uniform_log2k,
                                          fc_log2k=fc_log2k, kmaps=km)
    for l in layers:
        got = nw.acts[l["dst"]][idx.tolist()].cpu().numpy()
        assert got.dtype == acts[l["dst"]].dtype, l["name"]
        bad = int((got != acts[l["dst"]]).sum())
        assert bad == 0, "layer %s: %d of %d activations differ" % (l["name"], bad, got.size)
    assert np.allclose(logits[idx], ref_logits, rtol=1e-6, atol=0), "logits"


def test_tiny_resnet_uniform_k(psb, oracle):
    from workloads import build_network, tiny_resnet_layers

    L = tiny_resnet_layers()
    net = build_network(L, 40, 5, 2, 15, 15)
    ctx, nw, logits = _run_gpu(psb, L, net, 5, 1 << 3, seed=2, uniform_log2k=3)
    _compare(nw, logits, oracle, L, net, range(5), 2, 3)
    assert psb.PSB_PATH_TENSOR in nw.paths.values() and psb.PSB_PATH_SHIFT_ADD in nw.paths.values()
    nw.free(); ctx.close()


def test_batched_sampling_and_op_list_equal_the_layer_by_layer_calls(psb, oracle):
    """psb_sample_batch_run and psb_run must reproduce what the single calls give (and the oracle)."""
    import torch
    from paper_1904_02205_b200.network import Network
    from workloads import build_network, tiny_resnet_layers

    L = tiny_resnet_layers()
    net = build_network(L, 40, 3, 2, 15, 15)
    ctx = psb.Context(0)
    nw = Network(ctx, L, net, 3, 1 << 3, uniform_log2k=3)
    img = torch.from_numpy(net["image"][:3]).to(ctx.device)
    nw.sample(7)                      # layer by layer: creates the handles
    nw.forward(img)                   # layer by layer: records the paths
    nw.sample(11)                     # all layers in one batch, new seed
    logits = nw.forward(img).cpu().numpy()       # one psb_run call
    assert ctx.device_status() == 0
    for l in L:
        if l["op"] == "conv":
            got = ctx.weights_export(nw.weights[l["name"]], 3)[0].cpu().numpy().astype(np.int64)
            p = net["params"][l["name"]]
            assert np.array_equal(got, oracle.sample_level(p["w"], 11, p["layer_id"], 3)[0]), l["name"]
    _compare(nw, logits, oracle, L, net, range(3), 11, 3)
    nw.free(); ctx.close()


def test_tiny_resnet_per_location_draw_counts(psb, oracle):
    from workloads import build_network, saliency_kmaps, tiny_resnet_layers

    L = tiny_resnet_layers()
    net = build_network(L, 40, 6, 4, 15, 15)
    kmaps = saliency_kmaps(6, sorted({l["hout"] for l in L if l["op"] == "conv"}), 4, ref_res=10)
    ctx, nw, logits = _run_gpu(psb, L, net, 6, 0b11111, seed=4, uniform_log2k=3, fc_log2k=4, kmaps=kmaps)
    _compare(nw, logits, oracle, L, net, range(6), 4, 3, fc_log2k=4, kmaps=kmaps)
    nw.free(); ctx.close()


def test_tiny_mobilenet_pruned_8bit(psb, oracle):
    from workloads import build_network, tiny_mobilenet_layers

    L = tiny_mobilenet_layers()
    net = build_network(L, 32, 4, 3, 255, 127, prune_frac=0.5)
    ctx, nw, logits = _run_gpu(psb, L, net, 4, 1 << 4, seed=3, uniform_log2k=4)
    _compare(nw, logits, oracle, L, net, range(4), 3, 4)
    nw.free(); ctx.close()


def test_resnet50_batch64_k8_against_oracle_on_sampled_images(psb, oracle):
    """ResNet-50 shape, batch 64, k = 8, 4-bit activations, as the benchmark runs it; the oracle
    recomputes the first and the last image of the batch through all 54 layers."""
    from workloads import build_network, resnet50_layers

    L = resnet50_layers()
    net = build_network(L, 224, 64, 2, 15, 15)
    ctx, nw, logits = _run_gpu(psb, L, net, 64, 1 << 3, seed=2, uniform_log2k=3)
    _compare(nw, logits, oracle, L, net, [0, 63], 2, 3)
    nw.free(); ctx.close()


def test_mobilenetv2_batch64_k16_against_oracle_on_sampled_images(psb, oracle):
    from workloads import build_network, mobilenetv2_layers

    L = mobilenetv2_layers()
    net = build_network(L, 224, 64, 3, 255, 127, prune_frac=0.5)
    ctx, nw, logits = _run_gpu(psb, L, net, 64, 1 << 4, seed=3, uniform_log2k=4)
    _compare(nw, logits, oracle, L, net, [0, 31, 63], 3, 4)
    nw.free(); ctx.close()


def test_resnet50_batch128_adaptive_draw_counts(psb, oracle):
    """The adaptive run: per-location k in {1,2,4,8,16} (mean 4) from the seeded saliency field,
    classifier at k = 16, batch 128; oracle on one image."""
    from workloads import build_network, resnet50_layers, saliency_kmaps

    L = resnet50_layers()
    net = build_network(L, 224, 128, 4, 15, 15)
    kmaps = saliency_kmaps(128, [112, 56, 28, 14, 7], 4)
    frac = np.bincount(kmaps[56].ravel(), minlength=5) / kmaps[56].size
    assert np.allclose(frac, [0.30, 0.25, 0.25, 0.125, 0.075], atol=0.01)
    ctx, nw, logits = _run_gpu(psb, L, net, 128, 0b11111, seed=4, uniform_log2k=3, fc_log2k=4, kmaps=kmaps)
    _compare(nw, logits, oracle, L, net, [77], 4, 3, fc_log2k=4, kmaps=kmaps)
    nw.free(); ctx.close()
