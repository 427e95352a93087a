"""B200-native beam-shared Gated DeltaNet decode (placeholder until the binding lands)."""
