"""CPU oracle for CAT -- test infrastructure only (see cat_oracle.py)."""
