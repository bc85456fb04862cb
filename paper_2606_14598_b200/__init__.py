"""B200-native fused W8A8 linear layer (per-token int8 activations x per-channel int8 weights)."""
