"""B200-native fused LM-head + Confidence-Adaptive Token (CAT) weighted cross-entropy."""
