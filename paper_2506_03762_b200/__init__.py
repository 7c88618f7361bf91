"""B200-native AhaKV eviction step (score -> select -> compact) behind a C ABI."""
