"""SSD head-decoupled compressed KV cache: B200 (sm_100a) decode hot path behind a C ABI.

``binding`` (ctypes over ``libssd_b200.so``) is the product; ``workloads`` only draws seeded
synthetic inputs.  Nothing here falls back to a CPU implementation.
"""
__all__ = ["binding", "workloads", "build", "dist"]
