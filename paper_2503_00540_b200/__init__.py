"""B200-native retrieval hot path for in-context video KV-cache retrieval (ReKV)."""
