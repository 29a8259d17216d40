"""HashAttention decode path for NVIDIA B200 (sm_100a): ENCODE -> SCORE -> TOPK -> GATHER-ATT.

`workloads` holds the seeded synthetic input generators; `binding` is the thin ctypes layer over
the C-ABI CUDA library (loaded on first use; there is no CPU fallback)."""
__all__ = ["workloads", "binding"]
