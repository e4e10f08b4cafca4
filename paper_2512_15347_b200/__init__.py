"""B200-native hot path of the Pro-GRPO Expand-and-Prune rollout.

The product is the C-ABI library built from ``csrc/`` (declared in ``include/progrpo.h``);
``binding`` marshals torch tensors into it, ``rollout`` is a thin driver that owns device
buffers and streams, ``workloads`` holds the seeded synthetic inputs.
"""
__all__ = ["binding", "rollout", "workloads", "build"]
