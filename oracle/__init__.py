"""CPU checker for the CUDA library.  Test infrastructure only; see mdi_oracle.py."""
