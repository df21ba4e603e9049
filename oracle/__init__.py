"""CPU oracle of the PBT hot path (test infrastructure; never used by the GPU library)."""
