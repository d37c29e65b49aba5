"""B200-native G-KV decode-time KV-cache eviction: Python binding of the C-ABI library."""
