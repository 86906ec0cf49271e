"""CPU oracle for the RaZeR matmul path: test infrastructure only (see razer_oracle.py)."""
