// ef_lora_linear: Y = X @ W + alpha * (X @ A) @ Bm, tensor-core bound at large M.
//
// The form the paper's search selects for LoRA (Section 7.2): the low-rank projection T = alpha * (X @ A) is
// computed ONCE and stored ([M,16] bf16 in the workspace) instead of being recomputed per output tile, and the
// rank-16 update enters the main contraction as one extra K slab: Y = [X | T] @ [W ; Bm].  Both steps run in one
// launch: the grid has one block per SM, the blocks that have no output tile (or, if all have one, the last 16)
// compute T's 128-row pieces first and publish each with a release store; a tile's producer acquires the pieces it
// needs right before its last k block, ~40 us later on the benchmark shape, so T costs nothing on the critical path.
// (For M <= 16 the two steps are two launches of the weight-streaming skinny kernel instead.)
// Everything runs on tcgen05: TMA stages 128B-swizzled bf16 tiles in shared memory, one elected thread issues
// tcgen05.mma (kind::f16, bf16 operands, fp32 accumulators in TMEM), the epilogue warps read the accumulators back
// with tcgen05.ld.
//
// Refinement (Table 1): "MN" -- grid over output tiles, K traversed by the in-block loop.
//
// Operand layouts.  X tiles are K-major (K contiguous), W / Bm / A tiles are MN-major (N
// contiguous) exactly as they sit in global memory; the UMMA descriptors carry the major-ness, so
// nothing is transposed.
#include "host.cuh"
#include "ptx.cuh"

namespace ef {
namespace lora {

constexpr int kBM = 128, kBK = 64;
constexpr int kRank = 16;

// --------------------------------------------------------------------------------------------
// main kernel
// --------------------------------------------------------------------------------------------
constexpr int kBN = 256;
constexpr int kABytes = kBM * kBK * 2;            // 16 KiB: [128 rows][64 k] K-major, 128B swizzle
constexpr int kBAtomBytes = kBK * 128;            //  8 KiB: [64 k][64 n] MN-major, 128B swizzle
constexpr int kBBytes = (kBN / 64) * kBAtomBytes; // 32 KiB
constexpr int kThreads = 192;                     // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr uint32_t kTmemCols = 512;
// MT = 128-row sub-tiles per block tile.  MT = 1: 128x256 tiles, 4 stages of 48 KiB, two 256-column accumulators
// (the epilogue of one tile overlaps the mainloop of the next).  MT = 2: 256x256 tiles, 3 stages of 64 KiB, one
// accumulator of 2 x 256 columns: a third less operand traffic from L2 per flop (the mainloop is bound by the
// L2 -> shared-memory stream, not by the tensor pipe), no epilogue overlap.
template <int MT> struct MainCfg {
    static constexpr int kStages = MT == 1 ? 4 : 3;
    static constexpr int kStageBytes = MT * kABytes + kBBytes;
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + 256;
    static constexpr int kAccBufs = MT == 1 ? 2 : 1;
};

struct MainParams {
    __nv_bfloat16* Y;
    int M, N;
    int tiles_m, num_tiles;
    int k_blocks;   // K / 64
    int has_lora;   // 1: one more K block taken from (T, Bm)
    // T = alpha * X @ A is computed INSIDE this kernel by its last t_blocks blocks before they take output tiles
    // (on the benchmark shape those blocks have no tile at all: 128 tiles, 148 SMs), 128 rows at a time; every
    // finished 128-row piece is published by the last of its four epilogue warps (flags[2*piece]: arrivals, back to
    // zero; flags[2*piece+1] = epoch + 1), and a tile's producer waits for that value before it loads the T operand
    // of its last k block.  The last block to leave advances the epoch.
    int t_blocks, n_sub;       // blocks that compute T first; 128-row pieces of T
    float alpha;
    __nv_bfloat16* T;          // [m_pad][16]
    uint32_t* flags;           // [n_sub][2]
    uint32_t* epoch;           // [0] epoch, [1] blocks done
    uint32_t* status;
};

template <int MT>
__global__ void __launch_bounds__(kThreads, 1)
lora_main_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                 const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmA, const MainParams p) {
    constexpr int kStages = MainCfg<MT>::kStages, kStageBytes = MainCfg<MT>::kStageBytes, kAccBufs = MainCfg<MT>::kAccBufs;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
    uint64_t* full = bars;                       // [kStages]  TMA -> MMA
    uint64_t* empty = bars + kStages;            // [kStages]  MMA -> TMA
    uint64_t* acc_full = bars + 2 * kStages;     // [2]        MMA -> epilogue
    uint64_t* acc_empty = bars + 2 * kStages + 2;  // [2]      epilogue -> MMA
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 4);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 4); }
        *abort_flag = 0u;
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();  // no global access above this line
    const int total_kb = p.k_blocks + p.has_lora;
    const uint32_t epoch = __ldcg(p.epoch);
    // this block's share of T: pieces tb, tb + t_blocks, ... (none if it is not one of the last t_blocks blocks)
    const int tb = static_cast<int>(blockIdx.x) - (static_cast<int>(gridDim.x) - p.t_blocks);
    constexpr int kTBBytes = kBK * kRank * 2;   // 2 KiB: [64 k][16 r] MN-major, 32B swizzle

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmW);
            if (p.has_lora) { tma_prefetch_desc(&tmT); tma_prefetch_desc(&tmB); }
            tma_prefetch_desc(&tmA);
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            if (tb >= 0) {
                for (int sub = tb; sub < p.n_sub && ok; sub += p.t_blocks) {
                    for (int kb = 0; kb < p.k_blocks; ++kb) {
                        if (!mbar_wait(&empty[stage], phase ^ 1u, abort_flag, p.status, 1)) { ok = false; break; }
                        uint8_t* sA = smem + stage * kStageBytes;
                        mbar_expect_tx(&full[stage], kABytes + kTBBytes);
                        tma_load_2d(sA, &tmX, &full[stage], kb * kBK, sub * kBM);
                        tma_load_2d(sA + kABytes, &tmA, &full[stage], 0, kb * kBK);
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
                const int m0 = (tile % p.tiles_m) * (MT * kBM), n0 = (tile / p.tiles_m) * kBN;
                for (int kb = 0; kb < total_kb; ++kb) {
                    if (!mbar_wait(&empty[stage], phase ^ 1u, abort_flag, p.status, 1)) { ok = false; break; }
                    uint8_t* sA = smem + stage * kStageBytes;
                    uint8_t* sB = sA + MT * kABytes;
                    mbar_expect_tx(&full[stage], kStageBytes);
                    if (kb < p.k_blocks) {
#pragma unroll
                        for (int h = 0; h < MT; ++h) tma_load_2d(sA + h * kABytes, &tmX, &full[stage], kb * kBK, m0 + h * kBM);
#pragma unroll
                        for (int j = 0; j < kBN / 64; ++j)
                            tma_load_2d(sB + j * kBAtomBytes, &tmW, &full[stage], n0 + 64 * j, kb * kBK);
                    } else {  // rank-16 slab: columns >= 16 of T and rows >= 16 of Bm are out of bounds -> zero
                        // the pieces of T this tile reads were written by other blocks of this launch: wait for them
                        // (bounded), then order the generic-proxy observation before the async-proxy reads
                        for (int h = 0; h < MT && ok; ++h) {
                            const int sub = m0 / kBM + h;
                            if (sub >= p.n_sub) break;
                            const uint32_t want = epoch + 1u;
                            const unsigned long long t0 = globaltimer_ns();
                            uint32_t spins = 0;
                            while (ld_acquire_u32(&p.flags[2 * sub + 1]) != want) {
                                if ((++spins & 0xFFu) == 0u && (*abort_flag || globaltimer_ns() - t0 > kWaitLimitNs)) {
                                    *abort_flag = 1u;
                                    atomicCAS(p.status, 0u, kStatusTimeout | 7u);
                                    ok = false;
                                    break;
                                }
                            }
                        }
                        if (!ok) break;
                        fence_proxy_async_all();
#pragma unroll
                        for (int h = 0; h < MT; ++h) tma_load_2d(sA + h * kABytes, &tmT, &full[stage], 0, m0 + h * kBM);
#pragma unroll
                        for (int j = 0; j < kBN / 64; ++j)
                            tma_load_2d(sB + j * kBAtomBytes, &tmB, &full[stage], n0 + 64 * j, 0);
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(kBM, kBN, 0, 1);
            int stage = 0; uint32_t phase = 0;
            int iter = 0;
            bool ok = true;
            if (tb >= 0) {   // T pieces first: M128 N16 accumulators in the first columns of the accumulator buffer
                constexpr uint32_t idesc_t = make_idesc_bf16(kBM, kRank, 0, 1);
                for (int sub = tb; sub < p.n_sub && ok; sub += p.t_blocks, ++iter) {
                    const int acc = kAccBufs == 2 ? (iter & 1) : 0;
                    const uint32_t acc_phase = kAccBufs == 2 ? ((iter >> 1) & 1) : (iter & 1);
                    if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, p.status, 2)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * kBN;
                    for (int kb = 0; kb < p.k_blocks; ++kb) {
                        if (!mbar_wait(&full[stage], phase, abort_flag, p.status, 3)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t sA = smem_u32(smem + stage * kStageBytes);
                        const uint64_t a_desc = make_smem_desc(sA, 16, 1024, kSwizzle128B);
                        const uint64_t b_desc = make_smem_desc(sA + kABytes, 16, 256, kSwizzle32B);
                        for (int kk = 0; kk < kBK / 16; ++kk)  // B advances 16 k-rows of 32 B = 512 B
                            umma_ss(d_tmem, a_desc + static_cast<uint64_t>(kk * 2), b_desc + static_cast<uint64_t>(kk * 32), idesc_t,
                                    (kb | kk) != 0 ? 1u : 0u);
                        umma_commit(&empty[stage]);
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                    if (ok) umma_commit(&acc_full[acc]);
                }
            }
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++iter) {
                const int acc = kAccBufs == 2 ? (iter & 1) : 0;
                const uint32_t acc_phase = kAccBufs == 2 ? ((iter >> 1) & 1) : (iter & 1);
                if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, p.status, 2)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kBN;
                for (int kb = 0; kb < total_kb; ++kb) {
                    if (!mbar_wait(&full[stage], phase, abort_flag, p.status, 3)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sA = smem_u32(smem + stage * kStageBytes);
                    const uint64_t b_desc = make_smem_desc(sA + MT * kABytes, kBAtomBytes, 1024, kSwizzle128B);
                    const int nk = (kb < p.k_blocks) ? kBK / 16 : kRank / 16;
#pragma unroll
                    for (int h = 0; h < MT; ++h) {
                        const uint64_t a_desc = make_smem_desc(sA + h * kABytes, 16, 1024, kSwizzle128B);
                        for (int kk = 0; kk < nk; ++kk) {
                            // A advances 16 k = 32 B inside the swizzled row; B advances 16 k-rows = 2048 B
                            umma_ss(d_tmem + h * kBN, a_desc + static_cast<uint64_t>(kk * 2), b_desc + static_cast<uint64_t>(kk * 128),
                                    idesc, (kb | kk) != 0 ? 1u : 0u);
                        }
                    }
                    umma_commit(&empty[stage]);
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(&acc_full[acc]);
            }
        }
    } else {
        const int q = warp & 3;  // TMEM lane quadrant this warp may read
        int iter = 0;
        bool live = true;
        if (tb >= 0) {
            for (int sub = tb; sub < p.n_sub; sub += p.t_blocks, ++iter) {
                const int acc = kAccBufs == 2 ? (iter & 1) : 0;
                const uint32_t acc_phase = kAccBufs == 2 ? ((iter >> 1) & 1) : (iter & 1);
                if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[acc], acc_phase, abort_flag, p.status, 4))) { live = false; break; }
                tc_fence_after();
                uint32_t r[16];
                tmem_ld16(tmem_base + acc * kBN + (static_cast<uint32_t>(q * 32) << 16), r);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[acc]);
                const int row = sub * kBM + q * 32 + lane;   // < m_pad: T is padded to whole pieces
                uint4 lo, hi;
                lo.x = pack_bf16x2(p.alpha * __uint_as_float(r[0]), p.alpha * __uint_as_float(r[1]));
                lo.y = pack_bf16x2(p.alpha * __uint_as_float(r[2]), p.alpha * __uint_as_float(r[3]));
                lo.z = pack_bf16x2(p.alpha * __uint_as_float(r[4]), p.alpha * __uint_as_float(r[5]));
                lo.w = pack_bf16x2(p.alpha * __uint_as_float(r[6]), p.alpha * __uint_as_float(r[7]));
                hi.x = pack_bf16x2(p.alpha * __uint_as_float(r[8]), p.alpha * __uint_as_float(r[9]));
                hi.y = pack_bf16x2(p.alpha * __uint_as_float(r[10]), p.alpha * __uint_as_float(r[11]));
                hi.z = pack_bf16x2(p.alpha * __uint_as_float(r[12]), p.alpha * __uint_as_float(r[13]));
                hi.w = pack_bf16x2(p.alpha * __uint_as_float(r[14]), p.alpha * __uint_as_float(r[15]));
                uint4* dst = reinterpret_cast<uint4*>(p.T + static_cast<size_t>(row) * kRank);
                dst[0] = lo; dst[1] = hi;
                __threadfence();   // the rows are visible before the flag moves
                __syncwarp();
                if (lane == 0) {
                    // the last of the four warps publishes the piece: ready word = epoch + 1 (a word left behind by an
                    // earlier call, of this or another shape, is at most the current epoch and can never match)
                    const uint32_t prev = atomicAdd(&p.flags[2 * sub], 1u);
                    if (prev == 3u) {
                        p.flags[2 * sub] = 0u;
                        __threadfence();
                        st_release_u32(&p.flags[2 * sub + 1], epoch + 1u);
                    }
                }
            }
        }
        for (int tile = blockIdx.x; live && tile < p.num_tiles; tile += gridDim.x, ++iter) {
            const int acc = kAccBufs == 2 ? (iter & 1) : 0;
            const uint32_t acc_phase = kAccBufs == 2 ? ((iter >> 1) & 1) : (iter & 1);
            const int m0 = (tile % p.tiles_m) * (MT * kBM), n0 = (tile / p.tiles_m) * kBN;
            const bool ok = __all_sync(0xffffffffu, mbar_wait(&acc_full[acc], acc_phase, abort_flag, p.status, 4));
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int h = 0; h < MT; ++h) {
                const int row = m0 + h * kBM + q * 32 + lane;
                const uint32_t taddr = tmem_base + (acc + h) * kBN + (static_cast<uint32_t>(q * 32) << 16);
                __nv_bfloat16* yrow = p.Y + static_cast<size_t>(row) * p.N + n0;
#pragma unroll 1
                for (int c = 0; c < kBN / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld32(taddr + c * 32, r);
                    tmem_wait_ld();
                    if (row < p.M) {
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            const int col = n0 + c * 32 + v * 8;
                            if (col + 8 <= p.N) {
                                uint4 o;
                                o.x = pack_bf16x2(__uint_as_float(r[v * 8 + 0]), __uint_as_float(r[v * 8 + 1]));
                                o.y = pack_bf16x2(__uint_as_float(r[v * 8 + 2]), __uint_as_float(r[v * 8 + 3]));
                                o.z = pack_bf16x2(__uint_as_float(r[v * 8 + 4]), __uint_as_float(r[v * 8 + 5]));
                                o.w = pack_bf16x2(__uint_as_float(r[v * 8 + 6]), __uint_as_float(r[v * 8 + 7]));
                                *reinterpret_cast<uint4*>(yrow + c * 32 + v * 8) = o;
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[acc]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0) {   // the last block to leave opens the next epoch of the T flags
        __threadfence();
        const uint32_t prev = atomicAdd(&p.epoch[1], 1u);
        if (prev == gridDim.x - 1) {
            p.epoch[1] = 0u;
            p.epoch[0] = epoch + 1u;
        }
    }
}

struct Plan {
    int tiles_m, tiles_n, m_pad, k_blocks;
    size_t t_off, tail_counters_off, tail_part_off, total;
};
inline Plan make_plan(int M, int K, int N) {
    Plan pl;
    pl.tiles_m = (M + kBM - 1) / kBM;
    pl.tiles_n = (N + kBN - 1) / kBN;
    pl.m_pad = pl.tiles_m * kBM;
    pl.k_blocks = K / kBK;
    // M <= 16 takes the skinny-M kernels: their per-n-tile arrival counters sit right behind the header (inside
    // the window ef_workspace_init clears), their partial slots at the end
    const bool skinny_tail = M <= skinny::kLoraTailMaxM;
    pl.tail_counters_off = kHeaderBytes;
    pl.t_off = kDataOffset;   // fixed: a workspace may serve calls of different shapes
    pl.tail_part_off = pl.t_off + ((static_cast<size_t>(pl.m_pad) * kRank * 2 + 255) & ~size_t(255));
    pl.total = pl.tail_part_off + (skinny_tail ? skinny::lora_tail_partials_bytes() : 0);
    return pl;
}

}  // namespace lora
}  // namespace ef

extern "C" {

size_t ef_lora_linear_workspace_bytes(int M, int K, int N, int R) {
    if (M <= 0 || K <= 0 || N <= 0 || R != ef::lora::kRank || K % ef::lora::kBK != 0) return 0;
    return ef::lora::make_plan(M, K, N).total;
}

ef_status ef_lora_linear(const void* X, const void* W, const void* A, const void* Bm, void* Y, int M, int K, int N, int R,
                         float alpha, void* ws, size_t ws_bytes, void* stream) {
    using namespace ef;
    if (!X || !W || !A || !Bm || !Y) return EF_ERR_NULL;
    if (M <= 0 || K <= 0 || N <= 0 || R <= 0) return EF_ERR_SHAPE;
    if (R != lora::kRank || K % lora::kBK != 0 || N % 8 != 0) return EF_ERR_UNSUPPORTED;
    if (2 * ((M + lora::kBM - 1) / lora::kBM) > static_cast<int>(kMaxCounters)) return EF_ERR_UNSUPPORTED;
    if (!aligned(X, 16) || !aligned(W, 16) || !aligned(A, 16) || !aligned(Bm, 16) || !aligned(Y, 16)) return EF_ERR_ALIGN;
    if (!ws || ws_bytes < ef_lora_linear_workspace_bytes(M, K, N, R)) return EF_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return EF_ERR_ALIGN;
    DeviceInfo di;
    if (!current_device_info(&di)) return EF_ERR_CUDA;
    if (di.cc_major != 10) return EF_ERR_ARCH;
    const lora::Plan pl = lora::make_plan(M, K, N);
    uint8_t* w = static_cast<uint8_t*>(ws);
    __nv_bfloat16* T = reinterpret_cast<__nv_bfloat16*>(w + pl.t_off);

    CUtensorMap tmX, tmW, tmT, tmB, tmA;
    ef_status st;
    {
        const uint64_t dims[2] = {static_cast<uint64_t>(K), static_cast<uint64_t>(M)};
        const uint64_t strides[1] = {static_cast<uint64_t>(K) * 2};
        const uint32_t box[2] = {64, lora::kBM};
        if ((st = encode_tmap_bf16(&tmX, X, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    }
    {
        const uint64_t dims[2] = {static_cast<uint64_t>(N), static_cast<uint64_t>(K)};
        const uint64_t strides[1] = {static_cast<uint64_t>(N) * 2};
        const uint32_t box[2] = {64, lora::kBK};
        if ((st = encode_tmap_bf16(&tmW, W, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    }
    {
        const uint64_t dims[2] = {lora::kRank, static_cast<uint64_t>(pl.m_pad)};
        const uint64_t strides[1] = {lora::kRank * 2};
        const uint32_t box[2] = {64, lora::kBM};
        if ((st = encode_tmap_bf16(&tmT, T, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    }
    {
        const uint64_t dims[2] = {static_cast<uint64_t>(N), lora::kRank};
        const uint64_t strides[1] = {static_cast<uint64_t>(N) * 2};
        const uint32_t box[2] = {64, lora::kBK};
        if ((st = encode_tmap_bf16(&tmB, Bm, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    }
    {
        const uint64_t dims[2] = {lora::kRank, static_cast<uint64_t>(K)};
        const uint64_t strides[1] = {lora::kRank * 2};
        const uint32_t box[2] = {lora::kRank, lora::kBK};
        if ((st = encode_tmap_bf16(&tmA, A, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_32B)) != EF_OK) return st;
    }
    static bool attr_set[64] = {};
    if (!attr_set[di.device]) {
        EF_CUDA_CHECK(cudaFuncSetAttribute(lora::lora_main_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, lora::MainCfg<1>::kSmemBytes));
        EF_CUDA_CHECK(cudaFuncSetAttribute(lora::lora_main_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, lora::MainCfg<2>::kSmemBytes));
        attr_set[di.device] = true;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (M <= skinny::kLoraTailMaxM) {
        // Few rows: both kernels are weight-streaming problems, not tensor-bound ones.  Same two-kernel form
        // (T stored once, reused by every output tile), on the skinny-projection kernel.
        if (kHeaderBytes + skinny::lora_tail_counters_bytes(N) > kDataOffset) return EF_ERR_UNSUPPORTED;   // counters must lie in the init window
        uint32_t* status = reinterpret_cast<uint32_t*>(w);
        uint32_t* counters = reinterpret_cast<uint32_t*>(w + pl.tail_counters_off);
        float* partials = reinterpret_cast<float*>(w + pl.tail_part_off);
        if ((st = skinny::launch_lora_head(X, A, T, M, K, alpha, status, counters, partials, di, s)) != EF_OK) return st;
        return skinny::launch_lora_tail(X, W, T, Bm, Y, M, K, N, status, counters, partials, di, s);
    }
    {
        lora::MainParams mp;
        mp.Y = static_cast<__nv_bfloat16*>(Y);
        mp.M = M; mp.N = N;
        // 256-row block tiles (a third less operand traffic per flop) unless that costs more waves of the grid
        const int tiles1 = pl.tiles_m * pl.tiles_n, tm2 = (M + 2 * lora::kBM - 1) / (2 * lora::kBM), tiles2 = tm2 * pl.tiles_n;
        const int waves1 = (tiles1 + di.num_sms - 1) / di.num_sms, waves2 = (tiles2 + di.num_sms - 1) / di.num_sms;
        const int mt = (M > lora::kBM && 2 * waves2 <= waves1) ? 2 : 1;
        mp.tiles_m = mt == 2 ? tm2 : pl.tiles_m;
        mp.num_tiles = mp.tiles_m * pl.tiles_n;
        mp.k_blocks = pl.k_blocks; mp.has_lora = 1;
        mp.status = reinterpret_cast<uint32_t*>(w);
        // T = alpha * X @ A inside the same launch: the grid always has #SMs blocks (all resident at once, one per
        // SM), and the last t_blocks of them compute T's 128-row pieces before they look for output tiles.
        mp.alpha = alpha;
        mp.T = T;
        mp.flags = reinterpret_cast<uint32_t*>(w + kCounterOffset);
        mp.epoch = reinterpret_cast<uint32_t*>(w + 64);
        mp.n_sub = pl.tiles_m;
        const int grid = di.num_sms;
        int idle = grid - mp.num_tiles;
        if (idle < 0) idle = 0;
        mp.t_blocks = idle >= 4 ? idle : (grid < 16 ? grid : 16);   // idle blocks if there are some, else the last 16
        if (mp.t_blocks > mp.n_sub) mp.t_blocks = mp.n_sub;
        if (mt == 2)
            EF_CUDA_CHECK(launch_pdl(lora::lora_main_kernel<2>, dim3(grid), dim3(lora::kThreads), lora::MainCfg<2>::kSmemBytes, s,
                                     tmX, tmW, tmT, tmB, tmA, mp));
        else
            EF_CUDA_CHECK(launch_pdl(lora::lora_main_kernel<1>, dim3(grid), dim3(lora::kThreads), lora::MainCfg<1>::kSmemBytes, s,
                                     tmX, tmW, tmT, tmB, tmA, mp));
    }
    return EF_OK;
}

}  // extern "C"
