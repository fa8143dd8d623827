"""B200-native verification hot path of Spiffy (speculative decoding for
diffusion LLMs with calibrated draft graphs).

``paper_2509_18085_b200.spiffy`` is the binding of the C-ABI CUDA library
(``libspiffy.so``: spiffy_graph_attention, spiffy_unmask_decide,
spiffy_accept_walk); ``paper_2509_18085_b200.workloads`` draws the seeded
synthetic inputs.  Importing the package loads neither: the CUDA library is
opened on first use and that fails loudly when it has not been built.
"""
__all__ = ["spiffy", "workloads", "build"]
