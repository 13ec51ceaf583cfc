"""AVSG per-decode-step operator for B200 (sm_100a): C-ABI library + thin Python binding."""
