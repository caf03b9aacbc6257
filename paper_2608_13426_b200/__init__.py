"""B200-native hot path of Reduced Matrix Multiplication (RMM)."""
