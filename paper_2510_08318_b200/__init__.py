"""B200-native linear attention (Hedgehog feature map) behind a C-ABI library."""
