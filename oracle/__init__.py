"""CPU oracle for the grouped LM-head draft step: test infrastructure only."""
