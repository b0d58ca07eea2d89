"""B200-native routed attention of VORTA (full / sliding-tile / core-set per head)."""
