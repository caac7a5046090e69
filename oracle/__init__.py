"""CPU oracle for the MEDA compression pass.  Test infrastructure only: the product path never imports it."""
