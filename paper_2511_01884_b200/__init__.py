"""B200-native fused linear operator: Y = epilogue(act(X W^T + b)) with an optional row
reduction (sum, max, LayerNorm over N), as one hand-written sm_100a kernel per call."""
