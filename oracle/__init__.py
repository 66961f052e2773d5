"""Scalar CPU oracle of the batched CartPole step. Test infrastructure only."""
