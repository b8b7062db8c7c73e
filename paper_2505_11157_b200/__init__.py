"""Spherical neighborhood attention for B200 (sm_100a): forward and backward behind a C ABI."""
