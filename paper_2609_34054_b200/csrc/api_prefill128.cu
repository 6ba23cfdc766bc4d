// New-turn prefill attention kernels and their launch logic for head_dim 128.
#include "prefill_run.cuh"
PRECC_DEFINE_PREFILL_UNIT(128)
