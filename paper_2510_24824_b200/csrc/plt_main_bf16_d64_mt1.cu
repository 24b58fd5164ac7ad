#define PLT_INST_D 64
#define PLT_INST_MT 1
#define PLT_INST_NAME main_bf16_d64_mt1
#include "plt_main_bf16_inst.inl"
