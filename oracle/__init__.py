"""CPU oracle of the loss-MSE sensitivity pass: test infrastructure only."""
