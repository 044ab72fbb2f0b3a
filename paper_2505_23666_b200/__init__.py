"""B200-native LoLA per-layer attention step (sliding window + sparse cache + linear state)."""
__version__ = "0.1.0"
