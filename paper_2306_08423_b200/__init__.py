"""B200-native batched evaluation of DistSim's event-based activity timeline.

``workloads`` (seeded synthetic inputs) is pure numpy; the engine binding is
loaded on first use of ``paper_2306_08423_b200.engine`` and fails loudly when
the CUDA library has not been built.
"""
