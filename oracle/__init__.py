"""CPU oracle for the HTS-RL hot path.  Test infrastructure only: nothing in the
product package imports this."""
