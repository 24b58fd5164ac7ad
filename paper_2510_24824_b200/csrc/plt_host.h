// Host-side interface between the C-ABI layer and the kernel translation units.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>

#include "plt_common.cuh"

namespace plt {

// Variant of the bf16 main kernel.
struct MainVariant {
    int D, NT, RW;       // head dim, 8-row groups per warp, warps along the packed rows
    int HPC, KW, KS;     // KV heads per block, warps along the keys of a tile, 16-key slices per warp
    int tile_keys;       // keys per pipeline tile
    int stages;          // ring depth
    int grid;            // persistent blocks
    size_t smem;         // dynamic shared memory per block
    bool fp8;            // caches and windows hold E4M3 codes (the f16-product kernel)
};

// Opens a kernel's dynamic shared memory up to what the current device allows a block to opt in to. The attribute
// belongs to the function, not to a handle: several handles (and the allocation-free entry point) can share one
// kernel instance with different shared-memory sizes, so it is set to the device limit rather than to any one handle's
// size, which a later, smaller set-up would otherwise lower under an earlier handle. Each launch still passes its own size.
inline cudaError_t allow_max_dynamic_smem(const void* fn) {
    int dev = 0, optin = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) return e;
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, fn);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - (int)fa.sharedSizeBytes);
}

bool main_bf16_exists(int D, int NT, int RW, int HPC, int KW, int KS, bool fp8 = false);
size_t main_bf16_smem(int D, int NT, int RW, int HPC, int KW, int KS, int stages, int max_batch, bool fp8 = false);
// Keys per pipeline tile of a variant (0 if it does not exist): the warps along the keys split a tile or take turns.
int main_bf16_tile_keys(int D, int NT, int RW, int HPC, int KW, int KS, bool fp8 = false);
// Opens the kernel's shared-memory limit and reports how many blocks of this variant fit one SM.
cudaError_t main_bf16_prepare(const MainVariant& v, int* blocks_per_sm);
// overlap: launch with programmatic stream serialisation, so that this grid's set-up (which reads only what the caller
// passed) runs while the kernel before it in the stream (the pre-step kernel, or the merge kernel of the step before)
// finishes; the kernel waits for that kernel's completion before it reads or writes anything else.
cudaError_t launch_main_bf16(const MainVariant& v, const CUtensorMap maps[4], const Params& p, bool overlap,
                             cudaStream_t stream);

// fp32 SIMT main kernel (same plan, tile of kF32TileKeys keys, one KV head per block).
constexpr int kF32TileKeys = 32;
constexpr int kF32Threads = 256;
size_t main_f32_smem(int D, int R, int max_batch);
cudaError_t main_f32_prepare(int D, int R, int max_batch, int* blocks_per_sm);
cudaError_t launch_main_f32(const Params& p, int grid, size_t smem, cudaStream_t stream);

// tcgen05 / tensor-memory main kernel (bf16, d = 128, one KV head per item, 128-key tiles, one block per SM).
int main_umma_rows(int R);            // packed rows rounded up to the N of the instruction: 16, 32 or 64
int main_umma_max_slots();
size_t main_umma_smem(int R, int nslot, int max_batch);
cudaError_t main_umma_prepare(int R, size_t smem, int* blocks_per_sm);
cudaError_t launch_main_umma(const CUtensorMap maps[4], const Params& p, int grid, size_t smem, int nslot, int kbox,
                             int wbox, int cap, cudaStream_t stream);

// The same layout for E4M3 caches (tcgen05.mma kind::f8f6f4 on the codes, up to 32 packed rows; queries and
// probabilities as sums of E4M3 terms; hpc = 1 or 2 KV heads per work item, Params::hpc at launch). `qimg` / `qinv`: device scratch of max_batch * Hkv query images
// (main_umma_e4m3_image_bytes each) and as many floats, written by a pack kernel launched first.
int main_umma_e4m3_rows(int R);       // 16 or 32
int main_umma_e4m3_max_slots();     // ring slots of 16 KB: 4 for K tiles, the rest (3 to 6) for V tiles
int main_umma_e4m3_min_slots();
size_t main_umma_e4m3_smem(int R, int hpc, int nslot, int max_batch);
size_t main_umma_e4m3_image_bytes(int R);
cudaError_t main_umma_e4m3_prepare(int R, int hpc, bool half_pages, size_t smem, int* blocks_per_sm);
cudaError_t launch_pack_q_e4m3(const Params& p, uint8_t* qimg, float* qinv, cudaStream_t stream);
cudaError_t launch_main_umma_e4m3(const CUtensorMap maps[4], const Params& p, int grid, size_t smem, int nslot, int kbox,
                                  int wbox, int cap, const uint8_t* qimg, const float* qinv, cudaStream_t stream);

// Pre-step of a decode step: shared-cache append, window ring update, gate linear (writes through p.k_cache,
// p.v_cache, p.k_win, p.v_win, which the attention kernels only read).
cudaError_t launch_prestep(const Params& p, bool bf16, const void* k_new, const void* v_new, const float* w_gate,
                           const float* b_gate, float* gate_out, cudaStream_t stream);

cudaError_t launch_reduce(const Params& p, bool bf16, bool overlap, cudaStream_t stream);

}  // namespace plt
