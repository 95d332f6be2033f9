"""B200-native cloud-side verification step of edge-cloud speculative decoding.

`binding` loads the CUDA library (and raises if it is missing); `workloads`
draws seeded synthetic inputs and holds none of the method's arithmetic.
"""
__all__ = ["binding", "workloads", "build"]
