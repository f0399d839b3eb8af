"""AMXFP4 (arXiv 2411.09909) quantize + GEMM hot path for NVIDIA B200 (sm_100a).

`paper_2411_09909_b200.amx` is the thin binding over the C-ABI CUDA library;
`paper_2411_09909_b200.inputs` draws the seeded synthetic tensors.  Importing the
package loads nothing heavy; the CUDA library is opened on first use of `amx`.
"""
