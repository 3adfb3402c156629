"""B200-native MoE down-projection operator (grouped GEMM2 + GatherRS combine) with the
wave-quantized analytical selector of the communication-CTA count.

`binding` is the thin ctypes layer over the C-ABI library (argument marshalling only);
`workloads` makes seeded synthetic inputs.  The CUDA library is required: there is no CPU
or PyTorch fallback, and `binding` raises at first use when the library is missing.
"""

__all__ = ["binding", "workloads"]
