"""B200-native SAKI per-position routing."""
