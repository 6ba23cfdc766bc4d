// Decode attention kernels and their launch logic for head_dim 128.
#include "decode_run.cuh"
PRECC_DEFINE_DECODE_UNIT(128)
