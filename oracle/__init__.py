"""CPU oracle of the STAND hot path.  Test infrastructure only: see stand_oracle.cpp."""
