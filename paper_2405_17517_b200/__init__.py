"""B200-native WASH population operators (weight shuffle, PAPA EMA, final average)."""
