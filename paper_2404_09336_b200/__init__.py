"""Span-restricted decode attention for B200 (sm_100a): C-ABI library + binding."""
