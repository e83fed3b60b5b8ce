"""CPU oracle of the MoE layer forward pass (fp64, written from the paper).  Test infrastructure only."""
