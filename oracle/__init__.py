"""CPU checker for the SparsePR CUDA library.  Test infrastructure only."""
