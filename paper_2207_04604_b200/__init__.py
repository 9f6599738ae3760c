"""B200-native multiparty-BFV hot path of D2-MHE (arXiv 2207.04604).

`d2mhe` is the Python binding of the CUDA library (argument marshalling only);
`workloads` holds the seeded synthetic inputs and parameter presets.
"""
__all__ = ["d2mhe", "workloads"]
