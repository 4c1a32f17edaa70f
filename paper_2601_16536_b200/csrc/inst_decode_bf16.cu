#define W4A16_INST_BF true
#define W4A16_INST_NAME bf16
#include "inst_decode.cuh"
