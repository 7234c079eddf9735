"""B200-native recurrent-pipeline decoding (MDI-LLM hot path): Python binding of the C-ABI library."""
