"""TEST INFRASTRUCTURE: CPU oracle of the verify-and-feedback step (see sd_oracle.c)."""
