"""CPU oracle of the TriSpec verify pass: test infrastructure only (see trispec_oracle)."""
