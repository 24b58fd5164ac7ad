#define PLT_INST_D 128
#define PLT_INST_NT 2
#define PLT_INST_RW 2
#define PLT_INST_FP8 1
#define PLT_INST_NAME main_fp8_d128_n2r2
#include "plt_main_bf16_inst.inl"
