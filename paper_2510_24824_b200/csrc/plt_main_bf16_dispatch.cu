// Maps a bf16 main-kernel variant to the translation unit that instantiates it.
#include "plt_host.h"

namespace plt {

#define PLT_DECL(D, MT) \
    cudaError_t main_bf16_d##D##_mt##MT(int, const MainVariant&, const CUtensorMap*, const Params*, cudaStream_t, int*);
PLT_DECL(64, 1) PLT_DECL(64, 2) PLT_DECL(64, 4) PLT_DECL(128, 1) PLT_DECL(128, 2) PLT_DECL(128, 4)
#undef PLT_DECL

static cudaError_t dispatch(int op, const MainVariant& v, const CUtensorMap* maps, const Params* p, cudaStream_t s,
                            int* out) {
#define PLT_GO(D_, MT_) \
    if (v.D == D_ && v.MT == MT_) return main_bf16_d##D_##_mt##MT_(op, v, maps, p, s, out);
    PLT_GO(64, 1) PLT_GO(64, 2) PLT_GO(64, 4) PLT_GO(128, 1) PLT_GO(128, 2) PLT_GO(128, 4)
#undef PLT_GO
    return cudaErrorInvalidValue;
}

bool main_bf16_exists(int D, int MT, int HPC, int KW) {
    MainVariant v{D, MT, HPC, KW, 1, 1, 0};
    return dispatch(0, v, nullptr, nullptr, nullptr, nullptr) == cudaSuccess;
}

size_t main_bf16_smem(int D, int MT, int HPC, int KW, int stages, int max_batch) {
    MainVariant v{D, MT, HPC, KW, stages, max_batch, 0};
    int out = 0;
    if (dispatch(3, v, nullptr, nullptr, nullptr, &out) != cudaSuccess) return 0;
    return (size_t)out;
}

cudaError_t main_bf16_prepare(const MainVariant& v, int* blocks_per_sm) {
    return dispatch(1, v, nullptr, nullptr, nullptr, blocks_per_sm);
}

cudaError_t launch_main_bf16(const MainVariant& v, const CUtensorMap maps[4], const Params& p, cudaStream_t stream) {
    return dispatch(2, v, maps, &p, stream, nullptr);
}

}  // namespace plt
