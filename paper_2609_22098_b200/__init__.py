"""B200-native hot path of one TreeSpark round: Markov-head scoring with sibling sampling,
calibrated best-first tree expansion, and lossless tree verification, as CUDA kernels behind a
C ABI (``ts_score_parents``, ``ts_expand_tree``, ``ts_verify_tree``).

``synth`` makes the seeded inputs; ``binding`` marshals torch device pointers into the C ABI.
The compiled library is loaded on first use of ``binding`` and its absence is an error: there is
no CPU fallback.
"""
