"""Plain CPU oracle of the AWEQ calibration pass (test infrastructure only)."""
