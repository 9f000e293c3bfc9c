"""B200-native QESGD hot path: encode / decode-average-apply / logistic SGD step."""
