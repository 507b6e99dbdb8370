"""B200-native drop planner of PARD (proactive request dropping).

`binding` wraps the C-ABI CUDA library (libpard.so, built by `build`);
`inputs` draws the seeded synthetic workloads.  Importing the package loads
nothing; the library is opened at the first binding call and there is no
fallback when it is missing.
"""
__all__ = ["binding", "build", "inputs"]
