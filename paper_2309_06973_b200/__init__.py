"""B200-native pruning hot path: threshold, mask, zero structures, keep propagation, compaction."""
