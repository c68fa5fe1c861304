"""B200-native per-rank MoE expert block (count+dispatch, permute+pad, fp8 grouped SwiGLU FFN, combine)."""
