"""CPU oracle of the delayed synchronous step -- test infrastructure only (see abs_oracle.py)."""
