"""B200-native hybrid decode attention (partials + LSE merge)."""
