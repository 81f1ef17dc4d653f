"""Placement-semantics sweep for B200: batched evaluation of the paper's memory
and communication derivation rules (Theorems 1-2), its correctness predicates
(Theorems 3-4) and composition rules (Theorems 6-7, Remark 4) over a design
space enumerated on the device, reduced to capacity-filtered Pareto frontiers.

``paper_2601_02311_b200.ps``     the binding of the CUDA library (fails loudly
                                   if the library has not been built)
``paper_2601_02311_b200.synth``  seeded synthetic inputs (no arithmetic)
``paper_2601_02311_b200.build``  compiles the library for sm_100a
"""
