"""fp64 CPU oracle for SANTA++ decode attention. TEST INFRASTRUCTURE ONLY."""
