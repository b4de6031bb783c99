"""In-hindsight int8 quantized layers for B200 (sm_100a).

`paper_2105_04246_b200.hq` is the Python face of the C-ABI library (same call names);
`synth` and `workloads` hold seeded inputs and layer shapes.  Importing the package
does not load the CUDA library; the first `hq` call does, and raises if it is missing.
"""
__all__ = ["hq", "synth", "workloads"]
