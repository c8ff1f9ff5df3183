"""Token Radius Attention hot path for B200 (sm_100a): thin Python binding over the C-ABI library."""
