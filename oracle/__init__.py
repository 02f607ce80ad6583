"""CPU oracle for the CaDDTree hot path.  TEST INFRASTRUCTURE ONLY: the product never imports it."""
