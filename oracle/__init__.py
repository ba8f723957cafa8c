"""CPU oracle for the tests -- TEST INFRASTRUCTURE ONLY; never imported by the product path."""
