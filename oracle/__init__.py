"""CPU oracle of the QESGD hot path.  Test infrastructure, not product code."""
