"""B200-native fused log-likelihood of the rank-r CP multi-token prediction head."""
