"""B200-native sample production/consumption path (actor rollout, replay ring,
staleness-bounded sampling, TD error, GAE) behind a C-ABI CUDA library.

``synth`` (workload shapes and seeded inputs) imports nothing heavy; the binding
in ``binding`` loads the CUDA library on first use and fails loudly without it.
"""
