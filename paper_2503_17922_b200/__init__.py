"""WindowKV prefill-time KV-cache window selection for B200 (sm_100a).

`binding`   ctypes face of the C-ABI library (wkv_score_windows, wkv_select_topk_windows,
            wkv_gather_kv, wkv_compress_group); the only implementation of the path.
`workloads` seeded synthetic inputs of the benchmark configurations.
`build`     compiles the library in-tree with nvcc.
"""
__all__ = ["binding", "workloads", "build", "replicas"]
