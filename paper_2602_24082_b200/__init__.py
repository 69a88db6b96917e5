"""Preference-packed attention (forward + backward) for B200 (sm_100a).

The CUDA library is loaded lazily by :mod:`paper_2602_24082_b200.binding`; importing the
package (for example to reach :mod:`workloads`) needs neither a GPU nor the built library.
"""
__all__ = ["binding", "workloads", "cost_model"]
