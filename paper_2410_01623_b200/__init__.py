"""Fira optimizer update (arXiv 2410.01623) as hand-written sm_100a CUDA kernels
behind a C-ABI library, with a thin ctypes binding.

`paper_2410_01623_b200.binding` loads the shared library and mirrors its entry
points; `paper_2410_01623_b200.workloads` draws the seeded synthetic inputs.
Nothing is loaded at package import."""
