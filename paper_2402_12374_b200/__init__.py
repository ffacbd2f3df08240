"""B200-native token-tree verification (tree-masked attention + Sequoia's Algorithm 2).

The CUDA library is loaded lazily by :mod:`paper_2402_12374_b200.binding`; importing the
package itself needs no GPU.  There is no CPU fallback: every call into the binding fails
loudly if the library is missing or no CUDA device is present.
"""
__all__ = ["binding", "workloads"]
