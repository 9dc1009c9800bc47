"""CPU oracle for HiF8 (test infrastructure; never imported by the CUDA library or its binding)."""
