"""B200-native routed-expert MoE layer (route, permute, grouped SwiGLU GEMMs, combine)."""
