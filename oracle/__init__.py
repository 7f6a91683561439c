"""CPU checker for the CKKS RNS primitive layer.  Test infrastructure only:
nothing in the product package imports this."""
