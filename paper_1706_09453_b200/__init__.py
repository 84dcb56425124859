"""B200 (sm_100a) forward pass of a feed-forward DNN with binary weights and activations."""
