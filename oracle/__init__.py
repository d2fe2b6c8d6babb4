"""fp64 CPU oracle of the composed-prefill hot path (test infrastructure only)."""
