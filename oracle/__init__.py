"""Float64 CPU oracle for DARK random-feature attention (test infrastructure, not product code)."""
