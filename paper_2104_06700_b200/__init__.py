"""B200-native aggregation primitive (AP) of full-batch GraphSAGE training (DistGNN)."""
