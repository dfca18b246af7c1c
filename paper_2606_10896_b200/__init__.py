"""Flash-GMM hot path for B200: fused EM iteration of a diagonal-covariance Gaussian mixture.

``paper_2606_10896_b200.flashgmm`` is the binding of the C-ABI library (it raises if the CUDA library is missing);
``paper_2606_10896_b200.synth`` holds the seeded input generators.  Nothing is imported eagerly so that the input
generators stay usable on a machine without the compiled library.
"""

__all__ = ["flashgmm", "synth", "build"]
