"""libfopd: B200-native fused loss path of freshness-aware on-policy distillation."""
