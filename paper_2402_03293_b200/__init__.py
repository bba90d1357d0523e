"""Flora (arXiv 2402.03293) compress / accumulate / decompress hot path for NVIDIA B200 (sm_100a).

The CUDA library is loaded lazily by :mod:`paper_2402_03293_b200.binding`; importing the
package itself needs no GPU.  There is no CPU fallback: calling an operation without the
built CUDA library raises.
"""
__all__ = ["binding", "workloads", "hostlogic", "replicas"]
