"""CPU oracle of the KVCapsule decode path: test infrastructure only (see kvcapsule_oracle)."""
