"""signSGD / Signum with majority vote on B200: sign packing, bit-sliced majority vote and
the Signum parameter update as hand-written sm_100a kernels behind a C ABI.

``paper_1810_05291_b200.binding`` mirrors the C entry points one to one (argument
marshalling only); ``paper_1810_05291_b200.inputs`` generates the seeded synthetic
workloads; ``fusion``, ``optim`` and ``distributed`` put a model's tensors, a torch optimiser and
one worker per GPU on top of them. Importing the package does not load the CUDA library; the first call does,
and raises if the library has not been built.
"""

__all__ = ["binding", "inputs", "build"]
