"""CPU oracle (test infrastructure only; see reference.py)."""
