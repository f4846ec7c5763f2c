"""CPU oracle for the PPO learner step: test infrastructure, not product code."""
