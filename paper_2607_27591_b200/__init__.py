"""Prox decode-time sparse SwiGLU FFN for NVIDIA B200 (sm_100a).

`binding` wraps the C-ABI library libprox.so (include/prox.h); `inputs` makes
seeded synthetic workloads; `build` compiles the library.  Importing this
package does not load the library; `from paper_2607_27591_b200 import binding`
does, and fails if it has not been built.
"""
__all__ = ["binding", "inputs", "build"]
