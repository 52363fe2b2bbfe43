"""libspace: one auto-correct decoding step of SPACE (arXiv 2402.11809) on B200.

`paper_2402_11809_b200.binding` loads the CUDA library and mirrors its C entry
points; `paper_2402_11809_b200.workloads` generates the seeded synthetic
inputs.  Nothing is imported eagerly so that the input generators can be used
on a machine without the compiled library.
"""
__all__ = ["binding", "workloads", "build"]
