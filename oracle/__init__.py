"""CPU checker for the DSLA layer.  Test infrastructure: never imported by the product path."""
