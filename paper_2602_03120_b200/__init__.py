"""B200-native parameter pass of Quantized Evolution Strategies (perturb / update / replay)."""
