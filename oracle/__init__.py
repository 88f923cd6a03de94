"""CPU fp64 oracle (test infrastructure only; see ``reference.py``)."""
