"""Predictive delta coding of the KV cache for B200 (sm_100a): Python binding of libplc.so."""
