"""B200-native MoDSE (Mixture of Diverse Size Experts) feed-forward layer."""
