"""Seeded synthetic inputs shaped like the paper's workloads.

This package only *generates data*: filters, activations, per-channel constants,
draw-count maps and the lists of layers that make up the network-shaped
workloads.  It contains none of the method's arithmetic (no sampling, no
integer contraction) and is the one module shared by the CUDA tests, the
benchmark and the CPU oracle tests.

The paper evaluates on ImageNet / CIFAR-10 with pretrained weights (Sec. 4.2,
4.3); neither is available offline, so seeded tensors with the *shapes* of
those networks stand in for them.
"""
from .single import config1_fc, config2_conv  # noqa: F401
from .nets import (  # noqa: F401
    resnet50_layers, mobilenetv2_layers, build_network, saliency_kmaps, tiny_resnet_layers,
    tiny_mobilenet_layers, network_macs,
)
