"""B200-native PCG (Principled Coarse-Graining) group-level verification."""
