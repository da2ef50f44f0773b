"""B200-native decoder-layer engine (the compiled per-shard function of the Pathways workloads).

``paper_2203_12533_b200.binding`` is the ctypes binding over the C-ABI library
(``libpw.so``, built from ``csrc/``); ``paper_2203_12533_b200.inputs`` draws the
seeded synthetic workloads; ``data_parallel`` and ``pipeline_parallel`` are the
host plumbing of the multi-process forms (buffer handles and ordering only).
Importing the package loads nothing heavy.
"""
__all__ = ["binding", "inputs", "build", "data_parallel", "pipeline_parallel", "dispatch_study"]
