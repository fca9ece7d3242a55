"""B200-native bf16 scaled-dot-product attention (forward + backward) behind a C ABI.

``workloads`` holds the seeded synthetic inputs; ``binding`` marshals torch tensors into the
C entry points of ``libsdpa_b200.so`` (built by ``build``).  Importing the package loads nothing.
"""
__all__ = ["binding", "build", "workloads"]
