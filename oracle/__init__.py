"""CPU oracle: the plain fp64 definition of the GAS layer pass (test infrastructure only)."""
