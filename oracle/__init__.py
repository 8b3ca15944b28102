"""CPU oracle for the DeepCache hot path.  Test infrastructure only: never imported by the CUDA package."""
