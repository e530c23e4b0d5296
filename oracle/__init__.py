"""TEST INFRASTRUCTURE, NOT PRODUCT CODE: the CPU oracle of the quantized
convolution path.  Imported only by tests, the smoke check and the CPU-baseline
leg of the benchmark; the CUDA package never imports it."""
