// Pieces shared by the tcgen05 main kernels of the CLP decode attention (keys as the M dimension of
// tcgen05.mma): operand descriptors, bounded waits, the ring cursor, the warp reduction over a thread's rows and
// the walk that turns the tile plan into TMA box coordinates.
#pragma once
#include "plt_common.cuh"
#include "plt_ptx.cuh"

namespace plt {

namespace {

constexpr int UK = 128;                  // keys per tile
constexpr int UD = 128;                  // head dimension
constexpr int kSmThreads = 128;          // softmax threads
constexpr float kSlack = 8.f;
constexpr uint64_t kUmmaWaitNs = 1000000000ull;

// Shared-memory matrix descriptor of tcgen05.mma: start address, leading and stride byte offsets in
// 16-byte units, descriptor version 1, swizzle mode (0 = none, 2 = 128 bytes).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t swizzle) {
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | ((uint64_t)swizzle << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 A and B, majorness (0 = K-major, 1 = MN-major), N / 8, M / 16.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// The same for kind::f8f6f4 with E4M3 codes in A and B (format code 0 in both fields).
__host__ __device__ constexpr uint32_t instr_desc_e4m3(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

// Bounded wait that also gives up as soon as another thread of the block has given up.
__device__ __noinline__ bool wait_slow(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3fu) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kUmmaWaitNs) {
                *abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_test_wait(bar, parity)) return true;
    return wait_slow(bar, parity, abort_flag);
}

// Out-of-line step of the piece walk (the plan arithmetic is long once unrolled over the loops).
__device__ __noinline__ bool walk_next(PieceWalk& walk, Piece& pc, uint32_t& flags) { return walk.next_small(pc, flags); }

// Position in a ring of `size` slots: slot index and the parity of its current use.
struct Ring {
    int slot;
    uint32_t parity;
    __device__ Ring() : slot(0), parity(0) {}
    __device__ __forceinline__ void advance(int size) {
        if (++slot == size) {
            slot = 0;
            parity ^= 1u;
        }
    }
};

// Reduces N values per lane across the 32 lanes of a warp with N - 1 (+ a few) shuffles instead of 5 N: each
// step halves the values a lane still carries and doubles the lanes they cover. The result of row r goes to
// dst[r] (shared memory).
template <int N, bool MAX>
__device__ __forceinline__ void warp_reduce_rows(float (&v)[N], int lane, float* dst) {
    static_assert(N == 8 || N == 16 || N == 32 || N == 64, "rows per warp reduction");
    if constexpr (N == 64) {
        float a[32], b[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            a[i] = v[i];
            b[i] = v[32 + i];
        }
        warp_reduce_rows<32, MAX>(a, lane, dst);
        warp_reduce_rows<32, MAX>(b, lane, dst + 32);
    } else {
        int n = N;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            if (n > 1) {
                const bool up = (lane & o) != 0;
                n >>= 1;
#pragma unroll
                for (int i = 0; i < N / 2; ++i) {
                    if (i < n) {
                        const float keep = up ? v[i + n] : v[i];
                        const float send = up ? v[i] : v[i + n];
                        const float got = __shfl_xor_sync(0xffffffffu, send, o);
                        v[i] = MAX ? fmaxf(keep, got) : keep + got;
                    }
                }
            } else {
                const float got = __shfl_xor_sync(0xffffffffu, v[0], o);
                v[0] = MAX ? fmaxf(v[0], got) : v[0] + got;
            }
        }
        // N = 32: lane l holds row l. N = 16: lanes 2r and 2r + 1 both hold row r. N = 8: lanes 4r .. 4r + 3.
        if (N == 32) dst[lane] = v[0];
        else if (N == 16) { if ((lane & 1) == 0) dst[lane >> 1] = v[0]; }
        else if ((lane & 3) == 0) dst[lane >> 2] = v[0];
    }
}

// Launch-time geometry (set by the host from the tensor maps it encoded).
struct UmmaGeom {
    int ring;        // slots in the K ring and in the V ring
    int kbox;        // keys per TMA box of the shared cache (min(128, page size or capacity))
    int wbox;        // keys per TMA box of a window (min(128, w))
    int cap;         // tiles each producer keeps in flight (issued, not landed) at most; <= ring
};

// TMA boxes of one tile: (key coordinate, outermost coordinate) per box, the same for K and V.
struct TileCoords {
    int nbox, box_keys, head;
    bool window;
    int c1[UK / 16], c3[UK / 16];
};

// Walks the tiles of a block's range in order and yields their box coordinates.
struct TileSource {
    PieceWalk walk;
    Piece pc;
    WinCursor cur;
    int t;
    bool have;
    __device__ TileSource(const Params& p, const int32_t* sp, int64_t lo, int64_t hi, const int32_t* lens)
        : walk(p, sp, lo, hi, lens), t(0), have(false) {
        pc.t0 = pc.t1 = 0;
        cur.l = 0;
        cur.key0 = 0;
    }
    __device__ __noinline__ void next(const Params& p, const UmmaGeom& geo, TileCoords& tc, uint32_t& flags) {
        if (!have || t == pc.t1) {
            have = walk_next(walk, pc, flags);
            t = pc.t0;
            if (pc.kind == 1) cur.seek(p, pc.sp, pc.t0);
        }
        tc.head = pc.hg;
        tc.window = pc.kind == 1;
        if (pc.kind == 0) {
            const int key0 = t * UK;
            tc.box_keys = geo.kbox;
            if (p.page_size > 0) {
                const int rem = pc.sp.cmax - key0;   // keys that hold data from key0 on (>= 1)
                tc.nbox = (min(rem, UK) + tc.box_keys - 1) / tc.box_keys;
                for (int i = 0; i < tc.nbox; ++i) {
                    const int key = key0 + i * tc.box_keys;
                    int page = p.page_table[(int64_t)pc.b * p.max_pages + key / p.page_size];
                    if (page < 0 || page >= p.num_pool_pages) {
                        flags |= kDevPageIdClamped;
                        page = page < 0 ? 0 : p.num_pool_pages - 1;
                    }
                    tc.c1[i] = key % p.page_size;
                    tc.c3[i] = page;
                }
            } else {
                tc.nbox = 1;
                tc.c1[0] = key0;
                tc.c3[0] = pc.b;
            }
        } else {
            tc.box_keys = geo.wbox;
            tc.nbox = 1;
            tc.c1[0] = cur.key0;
            tc.c3[0] = pc.b * (p.L - 1) + (cur.l - 1);
            cur.advance(p, pc.sp);
        }
        ++t;
    }
};

// Waits as a warp: `failed` (a wait of this warp ran out) stays warp-uniform, because the tensor-memory
// loads and stores that depend on it are warp-collective.
__device__ __noinline__ bool sm_wait_slow(uint64_t* bar, uint32_t parity, volatile int* abort_flag, bool failed) {
    bool bad = false;
    if (!failed) bad = !wait_or_abort(bar, parity, abort_flag);
    return __any_sync(0xffffffffu, failed || bad);
}
__device__ __forceinline__ bool sm_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, bool failed) {
    if (__all_sync(0xffffffffu, !failed && mbar_test_wait(bar, parity))) return false;
    return sm_wait_slow(bar, parity, abort_flag, failed);
}

}  // namespace

}  // namespace plt
