"""B200-native SQuant weight quantization (progressive CASE solver): Python binding package."""
