// Maps a bf16 main-kernel variant to the translation unit that instantiates it.
#include "plt_host.h"

namespace plt {

#define PLT_ALL(X, D) X(D, 1, 1) X(D, 2, 1) X(D, 3, 1) X(D, 4, 1) X(D, 2, 2) X(D, 3, 2) X(D, 4, 2)
#define PLT_DECL(D, NT, RW) \
    cudaError_t main_bf16_d##D##_n##NT##r##RW(int, const MainVariant&, const CUtensorMap*, const Params*, cudaStream_t, int*);
PLT_ALL(PLT_DECL, 64) PLT_ALL(PLT_DECL, 128)
#undef PLT_DECL
#define PLT_DECL8(D, NT, RW) \
    cudaError_t main_fp8_d##D##_n##NT##r##RW(int, const MainVariant&, const CUtensorMap*, const Params*, cudaStream_t, int*);
PLT_ALL(PLT_DECL8, 128)
#undef PLT_DECL8

static cudaError_t dispatch(int op, const MainVariant& v, const CUtensorMap* maps, const Params* p, cudaStream_t s,
                            int* out) {
#define PLT_GO(D_, NT_, RW_) \
    if (v.D == D_ && v.NT == NT_ && v.RW == RW_) return main_bf16_d##D_##_n##NT_##r##RW_(op, v, maps, p, s, out);
#define PLT_GO8(D_, NT_, RW_) \
    if (v.D == D_ && v.NT == NT_ && v.RW == RW_) return main_fp8_d##D_##_n##NT_##r##RW_(op, v, maps, p, s, out);
    if (v.fp8) {
        PLT_ALL(PLT_GO8, 128)
        return cudaErrorInvalidValue;
    }
    PLT_ALL(PLT_GO, 64) PLT_ALL(PLT_GO, 128)
#undef PLT_GO
#undef PLT_GO8
#undef PLT_ALL
    return cudaErrorInvalidValue;
}

bool main_bf16_exists(int D, int NT, int RW, int HPC, int KW, int KS, bool fp8) {
    MainVariant v{D, NT, RW, HPC, KW, KS, 0, 1, 1, 0, fp8};
    return dispatch(0, v, nullptr, nullptr, nullptr, nullptr) == cudaSuccess;
}

size_t main_bf16_smem(int D, int NT, int RW, int HPC, int KW, int KS, int stages, int max_batch, bool fp8) {
    MainVariant v{D, NT, RW, HPC, KW, KS, 0, stages, max_batch, 0, fp8};
    int out = 0;
    if (dispatch(3, v, nullptr, nullptr, nullptr, &out) != cudaSuccess) return 0;
    return (size_t)out;
}

int main_bf16_tile_keys(int D, int NT, int RW, int HPC, int KW, int KS, bool fp8) {
    MainVariant v{D, NT, RW, HPC, KW, KS, 0, 1, 1, 0, fp8};
    int out = 0;
    if (dispatch(4, v, nullptr, nullptr, nullptr, &out) != cudaSuccess) return 0;
    return out;
}

cudaError_t main_bf16_prepare(const MainVariant& v, int* blocks_per_sm) {
    return dispatch(1, v, nullptr, nullptr, nullptr, blocks_per_sm);
}

cudaError_t launch_main_bf16(const MainVariant& v, const CUtensorMap maps[4], const Params& p, bool overlap,
                             cudaStream_t stream) {
    return dispatch(overlap ? 5 : 2, v, maps, &p, stream, nullptr);
}

}  // namespace plt
