"""Seeded synthetic inputs for the benchmark and the tests (not part of the library).

`synth` draws random numbers and lays out structure only; `rollout_sim` plays the inference engine that
produced the rollouts (plain torch); `workload` assembles the named micro-batches from the two.
"""
