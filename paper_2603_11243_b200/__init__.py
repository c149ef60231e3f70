"""B200-native decision kernels for CTC-draft self-speculative decoding of LLM-based ASR.

`binding` exposes the C ABI of libssd (ssd_ctc_draft, ssd_entropy_gate, ssd_verify);
`synth` holds the seeded synthetic workloads; `build` compiles the library for sm_100a.
"""
__all__ = ["binding", "synth", "build"]
