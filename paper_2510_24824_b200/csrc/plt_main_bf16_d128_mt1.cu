#define PLT_INST_D 128
#define PLT_INST_MT 1
#define PLT_INST_NAME main_bf16_d128_mt1
#include "plt_main_bf16_inst.inl"
