"""CPU oracle of the GLANCE speculative round.  Test infrastructure: never imported by the CUDA path."""
