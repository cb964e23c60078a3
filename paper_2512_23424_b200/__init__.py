"""B200-native last-axis softmax / log-softmax / LayerNorm / RMSNorm."""
