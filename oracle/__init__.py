"""CPU oracle for the CoRun hot path (test infrastructure only; see oracle.py)."""
