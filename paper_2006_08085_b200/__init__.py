"""B200-native DeTAG step (decentralized gradient tracking with accelerated gossip).

``inputs`` draws seeded synthetic graphs, gossip matrices and objective data.
``binding`` marshals arguments to the C-ABI library ``libdetag.so`` built from ``csrc/``;
every step of the hot path runs in that library's CUDA kernels.  Importing this package
loads nothing; the library is opened on first use and a missing build raises.
"""
__all__ = ["inputs", "binding", "build"]
