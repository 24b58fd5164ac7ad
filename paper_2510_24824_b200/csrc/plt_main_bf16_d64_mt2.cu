#define PLT_INST_D 64
#define PLT_INST_MT 2
#define PLT_INST_NAME main_bf16_d64_mt2
#include "plt_main_bf16_inst.inl"
