"""B200-native quantized convolution path (int8, power-of-two scales) of
Settle et al., "Quantizing Convolutional Neural Networks for Low-Power
High-Throughput Inference Engines" (2018).

The CUDA library is loaded lazily by `paper_1805_07941_b200.binding`; importing
the package itself needs no GPU."""
