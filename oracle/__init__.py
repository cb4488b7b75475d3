"""CPU oracle of the PPO hot path -- test infrastructure, never imported by the product path."""
