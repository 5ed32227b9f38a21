"""libfsoftmax: last-dimension softmax for NVIDIA B200 (sm_100a) behind a C ABI."""
