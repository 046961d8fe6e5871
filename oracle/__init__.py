"""CPU oracle for the batched Render step (test infrastructure only; see mv_oracle.c)."""
