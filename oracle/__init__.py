"""Float64 CPU oracle (test infrastructure only; never imported by the CUDA library or its binding)."""
