"""B200-native decompression hot path of the Ecco 4x block format (see include/ecco.h)."""
