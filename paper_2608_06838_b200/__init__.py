"""B200-native chunkwise gated linear recurrence over sequence segments (StateFlow's hot path)."""
