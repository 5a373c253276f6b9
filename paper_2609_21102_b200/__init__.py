"""B200-native spectrally deflated matrix filter (deflated polar factor and deflated PSD projection)."""
