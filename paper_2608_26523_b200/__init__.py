"""B200-native chunked-prefill attention (the hot path of the VPP chunked-prefill pipeline).

`paper_2608_26523_b200.api` binds the C-ABI library (`libvpp_chunk_attn.so`, built from `csrc/`);
`paper_2608_26523_b200.workloads` draws seeded synthetic inputs.  There is no CPU fallback: the
binding raises if the CUDA library cannot be loaded.
"""
__all__ = ["api", "workloads"]
