"""CPU oracle for the DeepSqueeze node update: test infrastructure only."""
