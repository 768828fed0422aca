"""B200-native AlexNet training step with two-replica exchange-and-average."""
