"""B200-native block-sparse prefill attention (block selection + sparse attention with mean correction)."""
