"""CPU oracle of the deterministic fused-upcast linear layer. Test infrastructure only."""
