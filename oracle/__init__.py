"""CPU oracle for the Jacobi hot path.  Test infrastructure only: see jacobi_oracle.c."""
