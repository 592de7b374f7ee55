"""CPU oracle (test infrastructure only; the CUDA path never imports it)."""
