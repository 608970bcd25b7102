"""B200-native Spark Transformer decode path (statistical top-k, Spark FFN, Spark attention)."""
