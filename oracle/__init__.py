"""CPU oracle of the Qsparse-local-SGD synchronisation round (test infrastructure only)."""
