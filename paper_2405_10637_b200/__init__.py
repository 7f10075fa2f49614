"""B200-native decode-step attention for the layer-condensed KV cache (LCKV)."""
