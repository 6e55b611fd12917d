"""B200-native tree-verify path of a prune-then-graft speculative decoding step.

`workloads` draws seeded synthetic inputs; `binding` loads the CUDA library (libgraft.so, built
in-tree by `build`) and exposes its C entry points under the same names.  There is no CPU
fallback: importing `binding` without the built library raises.
"""
__all__ = ["workloads", "binding", "build"]
