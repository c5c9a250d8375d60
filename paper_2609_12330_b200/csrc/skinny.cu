// ef_rmsnorm_matmul and ef_gated_mlp: projections of a few (<= 16) token rows through large
// weight matrices.  Arithmetic intensity is 8..16 flop/byte, so both are HBM-bound: the job is to
// stream W once at full bandwidth; the tensor core only has to keep up.
//
// Swap-AB on tcgen05: the MMA computes D^T[n, m] = sum_k W[k, n] * X[m, k] with the 128 weight
// columns of a tile as the MMA M dimension (A operand = W tile exactly as it lies in memory,
// MN-major) and the <= 16 token rows as the MMA N dimension (B operand = X tile, K-major).  The
// accumulator is 128 TMEM lanes x 16 fp32 columns per weight matrix.
//
// Refinement (Table 1, MatMul "NK"): the (n-tile, k-block) grid is flattened n-major and cut into
// equal contiguous ranges, one per persistent block, so every SM streams the same number of
// bytes.  A block that owns only part of a tile's K range stores its fp32 partial (Collection);
// the block that arrives last sums the partials in block order (Reduce_+ over the parallel K
// axis, deterministic) and only then applies the pointwise epilogue -- SiLU(gate)*up is nonlinear,
// so it cannot be applied to partial sums; the RMSNorm row factor r_m is invariant along K and is
// applied at the same place (Table 1, factor motion), while gamma varies along K and is folded
// into the X operand when the block builds it.  The same kernel with both options on is the
// RMSNorm-MLP program: Y = SiLU(r (X gamma) Wg) * (r (X gamma) Wu) in one launch.
#include "host.cuh"
#include "ptx.cuh"

namespace ef {
namespace skinny {

constexpr int kBN = 128;                          // weight columns per tile = MMA M
constexpr int kBK = 64;
constexpr int kMaxM = 16;                         // token rows = MMA N
constexpr int kWAtomBytes = kBK * 128;            // 8 KiB: [64 k][64 n] MN-major, 128B swizzle
constexpr int kWBytes = 2 * kWAtomBytes;          // 16 KiB per weight matrix per k block
constexpr int kXBytes = kMaxM * kBK * 2;          // 2 KiB: [16 rows][64 k] K-major, 128B swizzle
constexpr int kThreads = 192;                     // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr int kMaxGrid = 256;
constexpr int kMiscBytes = 1024 + kMaxGrid * 4;   // barriers, flags, r_m, slot table, row-sum partials
constexpr int kMaxSmem = 227 * 1024;

struct Params {
    const __nv_bfloat16* X;
    const __nv_bfloat16* gamma;  // NORM only
    const __nv_bfloat16* beta;   // LayerNorm only
    __nv_bfloat16* Y;
    int M, K, N;
    int n_tiles, k_blocks, total_units;
    int base, rem;       // block c owns base + (c < rem) consecutive (tile, k block) units
    int stages;
    int lora;            // NW == 1, no norm: the last k block of every n tile is the rank-16 update (T, Bm tiles)
    int tile_n;          // weight columns per tile: 128, or 64 (only the first 64-column atom of a tile is loaded and its
                         // results are used; twice as many tiles, so that small calls can give every block a whole tile)
    int pair;            // 1: a stage holds TWO consecutive k blocks (weight boxes of 128 rows, 16 KiB each: the copy engine
                         // moves more per request); only when every range starts at an even k block and has even length
    int pdl_mode;        // programmatic dependent launch: 0 = let the next kernel start at once, wait for the previous one
                         // before the first global access; 1 = wait first, THEN let the next kernel start (so the next one
                         // may read this kernel's inputs without waiting); 2 = no wait except before the T tile is loaded
                         // (the kernel before is a mode-1 kernel that produces nothing else this one reads)
    float eps;
    float out_scale;     // NW == 1, no norm: the result is multiplied by this before rounding (1 elsewhere)
    uint32_t* status;
    uint32_t* counters;  // one per n tile, zero between calls
    float* partials;     // [grid][2][NW][16][128]
};

__device__ __forceinline__ int range_begin(int c, int base, int rem) { return c * base + min(c, rem); }
__device__ __forceinline__ int owner_of(int x, int base, int rem) {
    const int big = rem * (base + 1);
    return x < big ? x / (base + 1) : rem + (x - big) / base;
}
// (u = k blocks per partition unit: 2 when a stage holds two k blocks, else 1)
__device__ __forceinline__ int slot_of(int c, int tile, int base, int rem, int k_blocks, int u) {
    return 2 * c + ((u * range_begin(c, base, rem) / k_blocks) == tile ? 0 : 1);
}
// A block's range is a sequence of SEGMENTS, one per n tile it touches.  Only the first and the last can be partial
// (shared with the neighbouring blocks).  Processing order: the partial LAST segment first, then the rest in
// natural order -- both owners of a shared tile then reach it at the very start of the kernel, and the partial
// exchange, the arrival counter and the merging block's epilogue overlap with the streaming of the whole tiles
// instead of forming a serial tail after it.
struct Seg {
    int it0, it1;
};
__device__ __forceinline__ int seg_count(int it_begin, int it_end, int k_blocks) {
    return it_end > it_begin ? (it_end - 1) / k_blocks - it_begin / k_blocks + 1 : 0;
}
__device__ __forceinline__ Seg seg_of(int s, int nseg, int it_begin, int it_end, int k_blocks) {
    const bool rotate = nseg >= 2 && (it_end % k_blocks) != 0;
    const int k = rotate ? (s == 0 ? nseg - 1 : s - 1) : s;   // natural index of the s-th processed segment
    const int tile = it_begin / k_blocks + k;
    Seg g;
    g.it0 = max(it_begin, tile * k_blocks);
    g.it1 = min(it_end, (tile + 1) * k_blocks);
    return g;
}
__device__ __forceinline__ float silu(float z) { return z / (1.f + __expf(-z)); }

// NW = number of weight matrices sharing the X operand (1: RMSNorm+matmul, 2: gated MLP)
// NORM = 1: build the X operand as bf16(x * gamma) in shared memory and scale rows by r_m at the end (RMSNorm);
// NORM = 2: LayerNorm: the operand is bf16((x - mean) * gamma), r_m = rsqrt(var + eps), and one spare operand row
//           holds beta, so the MMA itself produces beta @ W, which the epilogue adds unscaled
template <int NW, int NORM>
__global__ void __launch_bounds__(kThreads, 1)
skinny_kernel(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
              const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmT, const Params p) {
    constexpr int kStageBytes = NW * kWBytes + (NORM ? 0 : kXBytes);
    constexpr uint32_t kAccCols = NW * kMaxM;          // fp32 columns per accumulator buffer
    constexpr uint32_t kTmemCols = 64;                 // two buffers of <= 32 columns
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int xg_bytes = NORM ? p.k_blocks * kXBytes : 0;
    uint8_t* xg = smem;                                // NORM: [k_blocks][2 KiB] persistent X operand
    uint8_t* stages = smem + xg_bytes;
    const int stage_bytes = p.pair ? 2 * kStageBytes : kStageBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(stages + p.stages * stage_bytes);
    uint64_t* full = bars;                             // [stages]
    uint64_t* empty = bars + p.stages;                 // [stages]
    uint64_t* acc_full = bars + 2 * p.stages;          // [2]
    uint64_t* acc_empty = bars + 2 * p.stages + 2;     // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * p.stages + 4);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    uint32_t* is_last = tmem_slot + 2;
    float* rinv = reinterpret_cast<float*>(tmem_slot + 4);        // [16]
    int* slot_table = reinterpret_cast<int*>(tmem_slot + 4 + kMaxM);  // [kMaxGrid]
    float* ssw = reinterpret_cast<float*>(slot_table + kMaxGrid);      // [5 warps][16 rows]
    float* mean = ssw + 5 * kMaxM;                                      // [16] LayerNorm row means

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr bool LN = (NORM == 2);
    // X operand as hi/lo row pairs (see the prologue); LayerNorm keeps row 7 (split) or 15 for beta
    const bool split = NORM && p.M <= (LN ? 7 : 8);
    const int beta_row = split ? 7 : 15;
    const int pu = p.pair ? 2 : 1;   // the partition counts pairs of k blocks when a stage holds two
    const int it_begin = pu * range_begin(blockIdx.x, p.base, p.rem);
    const int it_end = pu * range_begin(blockIdx.x + 1, p.base, p.rem);
    const int nseg = seg_count(it_begin, it_end, p.k_blocks);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 4); }
        *abort_flag = 0u;
        *is_last = 0u;
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
    if (p.pdl_mode != 1) pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (p.pdl_mode != 2) pdl_wait();  // everything below may touch global memory of the previous kernel in the stream
    if (p.pdl_mode == 1) pdl_launch_dependents();

    // The producer starts streaming W right away; everyone else first builds the X operand.
    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&tmW0);
            if (NW == 2) tma_prefetch_desc(&tmW1);
            if (!NORM) tma_prefetch_desc(&tmX);
            if (NW == 1 && !NORM && p.lora) { tma_prefetch_desc(&tmW1); tma_prefetch_desc(&tmT); }
            int stage = 0; uint32_t phase = 0;
            bool okp = true;
            bool t_waited = false;
            for (int sg = 0; sg < nseg && okp; ++sg) {
              const Seg seg = seg_of(sg, nseg, it_begin, it_end, p.k_blocks);
              const int tile = seg.it0 / p.k_blocks;
              for (int it = seg.it0; it < seg.it1; it += (p.pair ? 2 : 1)) {
                const int kb = it - tile * p.k_blocks;
                if (!mbar_wait(&empty[stage], phase ^ 1u, abort_flag, p.status, 1)) { okp = false; break; }
                uint8_t* st = stages + stage * stage_bytes;
                const bool wide = p.tile_n == kBN;
                mbar_expect_tx(&full[stage], stage_bytes - (wide ? 0 : NW * kWAtomBytes * (p.pair ? 2 : 1)));
                const int n0 = tile * p.tile_n, k0 = kb * kBK;
                if (p.pair && NW == 1 && !NORM && p.lora && kb == p.k_blocks - 2) {
                    // the rank-16 update as the last double stage: Bm rows 16..127 and T columns 16..127 lie outside their
                    // tensors and are filled with zeros (the second weight map carries Bm here, with 128-row boxes)
                    if (p.pdl_mode == 2 && !t_waited) { pdl_wait(); t_waited = true; }   // T comes from the kernel before
                    tma_load_2d(st, &tmW1, &full[stage], n0, 0);
                    if (wide) tma_load_2d(st + 2 * kWAtomBytes, &tmW1, &full[stage], n0 + 64, 0);
                    tma_load_2d(st + NW * 2 * kWBytes, &tmT, &full[stage], 0, 0);
                    tma_load_2d(st + NW * 2 * kWBytes + kXBytes, &tmT, &full[stage], 64, 0);
                } else if (p.pair) {
                    // two k blocks per stage: the weight maps carry boxes of 128 rows here; layout per weight matrix
                    // [n half 0: 128 k rows][n half 1: 128 k rows], then the two X tiles
                    tma_load_2d(st, &tmW0, &full[stage], n0, k0);
                    if (wide) tma_load_2d(st + 2 * kWAtomBytes, &tmW0, &full[stage], n0 + 64, k0);
                    if (NW == 2) {
                        tma_load_2d(st + 2 * kWBytes, &tmW1, &full[stage], n0, k0);
                        if (wide) tma_load_2d(st + 2 * kWBytes + 2 * kWAtomBytes, &tmW1, &full[stage], n0 + 64, k0);
                    }
                    if (!NORM) {
                        tma_load_2d(st + NW * 2 * kWBytes, &tmX, &full[stage], k0, 0);
                        tma_load_2d(st + NW * 2 * kWBytes + kXBytes, &tmX, &full[stage], k0 + kBK, 0);
                    }
                } else
                if (NW == 1 && !NORM && p.lora && kb == p.k_blocks - 1) {
                    // the rank-16 update as one more k block: Bm rows 16..63 and T columns 16..63 lie outside
                    // their tensors and are filled with zeros (the second weight map carries Bm here)
                    if (p.pdl_mode == 2 && !t_waited) { pdl_wait(); t_waited = true; }   // T comes from the kernel before
                    tma_load_2d(st, &tmW1, &full[stage], n0, 0);
                    if (wide) tma_load_2d(st + kWAtomBytes, &tmW1, &full[stage], n0 + 64, 0);
                    tma_load_2d(st + NW * kWBytes, &tmT, &full[stage], 0, 0);
                } else {
                    tma_load_2d(st, &tmW0, &full[stage], n0, k0);
                    if (wide) tma_load_2d(st + kWAtomBytes, &tmW0, &full[stage], n0 + 64, k0);
                    if (NW == 2) {
                        tma_load_2d(st + kWBytes, &tmW1, &full[stage], n0, k0);
                        if (wide) tma_load_2d(st + kWBytes + kWAtomBytes, &tmW1, &full[stage], n0 + 64, k0);
                    }
                    if (!NORM) tma_load_2d(st + NW * kWBytes, &tmX, &full[stage], k0, 0);
                }
                if (++stage == p.stages) { stage = 0; phase ^= 1u; }
              }
            }
        }
    } else if (NORM) {
        // X operand = bf16(x * gamma) for ALL k blocks, written in the K-major 128B-swizzled tile
        // layout the MMA descriptor expects (row r of a tile: 128 B, 16-byte chunk c stored at
        // chunk c ^ (r & 7)); sum of squares per row for r_m (product fusion: same pass over X).
        // Thread i of the 160 owns 16-byte column chunk i (+160, ...) of EVERY row: all of a thread's
        // loads are independent and issued together, so the whole prologue costs one memory latency.
        const int idx = threadIdx.x - 32;  // 0..159
        const int chunks = p.K >> 3;
        float ss[kMaxM];
        float mu[kMaxM];
#pragma unroll
        for (int r = 0; r < kMaxM; ++r) { ss[r] = 0.f; mu[r] = 0.f; }
        if (LN) {
            // row means first (a pass of its own: the deviations x - mean are what gets squared and multiplied)
            for (int c = idx; c < chunks; c += 160) {
#pragma unroll
                for (int r = 0; r < kMaxM; ++r) {
                    if (r < p.M) {
                        const uint4 xv = __ldg(reinterpret_cast<const uint4*>(p.X + static_cast<size_t>(r) * p.K) + c);
                        const uint32_t xs[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) mu[r] += __uint_as_float(xs[j] << 16) + __uint_as_float(xs[j] & 0xFFFF0000u);
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < kMaxM; ++r) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mu[r] += __shfl_xor_sync(0xffffffffu, mu[r], o);
                if (lane == 0) ssw[(warp - 1) * kMaxM + r] = mu[r];
            }
            asm volatile("bar.sync 2, 160;" ::: "memory");
            if (idx < kMaxM) {
                float tot = 0.f;
#pragma unroll
                for (int w = 0; w < 5; ++w) tot += ssw[w * kMaxM + idx];
                mean[idx] = tot / static_cast<float>(p.K);
            }
            asm volatile("bar.sync 2, 160;" ::: "memory");
#pragma unroll
            for (int r = 0; r < kMaxM; ++r) mu[r] = mean[r];
        }
        for (int c = idx; c < chunks; c += 160) {
            const uint4 gv = __ldg(reinterpret_cast<const uint4*>(p.gamma) + c);
            uint4 xv[kMaxM];
#pragma unroll
            for (int r = 0; r < kMaxM; ++r) {
                xv[r] = make_uint4(0u, 0u, 0u, 0u);
                if (r < p.M) xv[r] = __ldg(reinterpret_cast<const uint4*>(p.X + static_cast<size_t>(r) * p.K) + c);
            }
            const uint32_t gs[4] = {gv.x, gv.y, gv.z, gv.w};
            const int kb = c >> 3, cc = c & 7;
            if (split) {
                // M <= 8: rows 0..7 hold hi = bf16(x*gamma), rows 8..15 hold lo = bf16(x*gamma - hi); the MMA
                // produces both partial results at no extra cost and the epilogue adds them, so the X
                // operand effectively carries 16 mantissa bits (x and gamma are bf16: the product has 16).
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    const uint32_t xs[4] = {xv[r].x, xv[r].y, xv[r].z, xv[r].w};
                    uint32_t hi4[4], lo4[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float x0 = __uint_as_float(xs[j] << 16), x1 = __uint_as_float(xs[j] & 0xFFFF0000u);
                        if (LN && r < p.M) { x0 -= mu[r]; x1 -= mu[r]; }
                        const float g0 = __uint_as_float(gs[j] << 16), g1 = __uint_as_float(gs[j] & 0xFFFF0000u);
                        ss[r] += x0 * x0 + x1 * x1;
                        const float v0 = x0 * g0, v1 = x1 * g1;
                        hi4[j] = pack_bf16x2(v0, v1);
                        const float h0 = __uint_as_float(hi4[j] << 16), h1 = __uint_as_float(hi4[j] & 0xFFFF0000u);
                        lo4[j] = pack_bf16x2(v0 - h0, v1 - h1);
                    }
                    *reinterpret_cast<uint4*>(xg + kb * kXBytes + r * 128 + ((cc ^ (r & 7)) << 4)) =
                        make_uint4(hi4[0], hi4[1], hi4[2], hi4[3]);
                    *reinterpret_cast<uint4*>(xg + kb * kXBytes + (r + 8) * 128 + ((cc ^ (r & 7)) << 4)) =
                        make_uint4(lo4[0], lo4[1], lo4[2], lo4[3]);
                }
            } else {
#pragma unroll
                for (int r = 0; r < kMaxM; ++r) {
                    const uint32_t xs[4] = {xv[r].x, xv[r].y, xv[r].z, xv[r].w};
                    uint32_t outv[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float x0 = __uint_as_float(xs[j] << 16), x1 = __uint_as_float(xs[j] & 0xFFFF0000u);
                        if (LN && r < p.M) { x0 -= mu[r]; x1 -= mu[r]; }
                        const float g0 = __uint_as_float(gs[j] << 16), g1 = __uint_as_float(gs[j] & 0xFFFF0000u);
                        ss[r] += x0 * x0 + x1 * x1;
                        outv[j] = pack_bf16x2(x0 * g0, x1 * g1);
                    }
                    *reinterpret_cast<uint4*>(xg + kb * kXBytes + r * 128 + ((cc ^ (r & 7)) << 4)) =
                        make_uint4(outv[0], outv[1], outv[2], outv[3]);
                }
            }
            if (LN) {   // the spare row carries beta (exact in bf16); its partner lo row, if any, stays zero
                const uint4 bv = __ldg(reinterpret_cast<const uint4*>(p.beta) + c);
                *reinterpret_cast<uint4*>(xg + kb * kXBytes + beta_row * 128 + ((cc ^ (beta_row & 7)) << 4)) = bv;
                if (split)
                    *reinterpret_cast<uint4*>(xg + kb * kXBytes + 15 * 128 + ((cc ^ 7) << 4)) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        // per-row sum of squares: warp shuffle tree, then the five warp partials in warp order (deterministic)
#pragma unroll
        for (int r = 0; r < kMaxM; ++r) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ss[r] += __shfl_xor_sync(0xffffffffu, ss[r], o);
            if (lane == 0) ssw[(warp - 1) * kMaxM + r] = ss[r];
        }
        fence_proxy_async_smem();
        asm volatile("bar.sync 2, 160;" ::: "memory");
        if (idx < kMaxM) {
            float tot = 0.f;
#pragma unroll
            for (int w = 0; w < 5; ++w) tot += ssw[w * kMaxM + idx];
            rinv[idx] = rsqrtf(tot / static_cast<float>(p.K) + p.eps);
        }
    }
    if (NORM && warp != 0) asm volatile("bar.sync 2, 160;" ::: "memory");  // warps 1..5; the producer keeps streaming

    if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(kBN, kMaxM, 1, 0);  // A MN-major, B K-major
            int stage = 0; uint32_t phase = 0;
            int iter = 0;
            bool ok = true;
            for (int sg = 0; sg < nseg && ok; ++sg) {
                const Seg seg = seg_of(sg, nseg, it_begin, it_end, p.k_blocks);
                const int it = seg.it0, seg_end = seg.it1;
                const int tile = it / p.k_blocks;
                const int kb0 = it - tile * p.k_blocks;
                const int acc = iter & 1;
                if (!mbar_wait(&acc_empty[acc], ((iter >> 1) & 1) ^ 1u, abort_flag, p.status, 2)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kAccCols;
                for (int i = 0; i < seg_end - it; i += (p.pair ? 2 : 1)) {
                    if (!mbar_wait(&full[stage], phase, abort_flag, p.status, 3)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t st = smem_u32(stages + stage * stage_bytes);
                    if (p.pair) {
                        // 128 k rows per stage: eight K = 16 steps; the second X tile follows the first
                        const uint32_t xs = NORM ? smem_u32(xg + (kb0 + i) * kXBytes) : st + NW * 2 * kWBytes;
                        const uint64_t b_desc = make_smem_desc(xs, 16, 1024, kSwizzle128B);
#pragma unroll
                        for (int w = 0; w < NW; ++w) {
                            const uint64_t a_desc = make_smem_desc(st + w * 2 * kWBytes, 2 * kWAtomBytes, 1024, kSwizzle128B);
#pragma unroll
                            for (int kk = 0; kk < 2 * kBK / 16; ++kk)
                                umma_ss(d_tmem + w * kMaxM, a_desc + static_cast<uint64_t>(kk * 128),
                                        b_desc + static_cast<uint64_t>((kk >> 2) * (kXBytes >> 4) + (kk & 3) * 2), idesc,
                                        (i | kk) != 0 ? 1u : 0u);
                        }
                    } else {
                    const uint32_t xs = NORM ? smem_u32(xg + (kb0 + i) * kXBytes) : st + NW * kWBytes;
                    const uint64_t b_desc = make_smem_desc(xs, 16, 1024, kSwizzle128B);
#pragma unroll
                    for (int w = 0; w < NW; ++w) {
                        const uint64_t a_desc = make_smem_desc(st + w * kWBytes, kWAtomBytes, 1024, kSwizzle128B);
#pragma unroll
                        for (int kk = 0; kk < kBK / 16; ++kk)
                            umma_ss(d_tmem + w * kMaxM, a_desc + static_cast<uint64_t>(kk * 128),
                                    b_desc + static_cast<uint64_t>(kk * 2), idesc, (i | kk) != 0 ? 1u : 0u);
                    }
                    }
                    umma_commit(&empty[stage]);
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(&acc_full[acc]);
                ++iter;
            }
        }
    } else if (warp >= 2) {
        const int q = warp & 3;
        const int et = q * 32 + lane;  // 0..127: TMEM lane = weight column within the tile
        int iter = 0;
        for (int sg = 0; sg < nseg; ++sg) {
            const Seg seg = seg_of(sg, nseg, it_begin, it_end, p.k_blocks);
            const int it = seg.it0, seg_end = seg.it1;
            const int tile = it / p.k_blocks;
            const int kb0 = it - tile * p.k_blocks;
            const int tile_end = (tile + 1) * p.k_blocks;
            const bool whole = (kb0 == 0) && (seg_end == tile_end);
            const int acc = iter & 1;
            if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[acc], (iter >> 1) & 1, abort_flag, p.status, 4))) break;
            tc_fence_after();
            uint32_t v[NW][16];
#pragma unroll
            for (int w = 0; w < NW; ++w)
                tmem_ld16(tmem_base + acc * kAccCols + w * kMaxM + (static_cast<uint32_t>(q * 32) << 16), v[w]);
            tmem_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[acc]);  // accumulator is in registers now
            const int n = (et < p.tile_n) ? tile * p.tile_n + et : p.N;   // lanes beyond a 64-column tile hold nothing
            bool finish = whole;
            int n_parts = 0;
            if (!whole) {
                float* ps = p.partials + static_cast<size_t>(slot_of(blockIdx.x, tile, p.base, p.rem, p.k_blocks, pu)) * (NW * kMaxM * kBN);
#pragma unroll
                for (int w = 0; w < NW; ++w)
#pragma unroll
                    for (int m = 0; m < kMaxM; ++m) ps[(w * kMaxM + m) * kBN + et] = __uint_as_float(v[w][m]);
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                const int c_first = owner_of(tile * p.k_blocks / pu, p.base, p.rem);
                const int c_last = owner_of((tile_end - 1) / pu, p.base, p.rem);
                n_parts = c_last - c_first + 1;
                if (warp == 2 && lane == 0) {
                    const uint32_t prev = atomicAdd(&p.counters[tile], 1u);
                    *is_last = (prev == static_cast<uint32_t>(n_parts - 1)) ? 1u : 0u;
                }
                for (int i = threadIdx.x - 64; i < n_parts; i += 128)
                    slot_table[i] = slot_of(c_first + i, tile, p.base, p.rem, p.k_blocks, pu);
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (*is_last) {
                    __threadfence();
#pragma unroll
                    for (int w = 0; w < NW; ++w)
#pragma unroll
                        for (int m = 0; m < kMaxM; ++m) v[w][m] = 0u;
                    for (int i = 0; i < n_parts; ++i) {  // block order: deterministic
                        const float* src = p.partials + static_cast<size_t>(slot_table[i]) * (NW * kMaxM * kBN);
#pragma unroll
                        for (int w = 0; w < NW; ++w)
#pragma unroll
                            for (int m = 0; m < kMaxM; ++m)
                                v[w][m] = __float_as_uint(__uint_as_float(v[w][m]) + __ldcg(src + (w * kMaxM + m) * kBN + et));
                    }
                    finish = true;
                }
            }
            if (finish && n < p.N) {
#pragma unroll
                for (int m = 0; m < kMaxM; ++m) {
                    if (m < p.M) {
                        // r_m is invariant along K: it scales each finished projection (factor motion)
                        const float r = NORM ? rinv[m] : (NW == 1 ? p.out_scale : 1.f);
                        float a0 = __uint_as_float(v[0][m]), a1 = __uint_as_float(v[NW - 1][m]);
                        if (split) {  // hi + lo halves of the X operand (m < 8 here)
                            a0 += __uint_as_float(v[0][(m + 8) & 15]);
                            a1 += __uint_as_float(v[NW - 1][(m + 8) & 15]);
                        }
                        float y;
                        if (NW == 2) y = silu(a0 * r) * (a1 * r);
                        else y = a0 * r;
                        if (LN) y += __uint_as_float(split ? v[0][7] : v[0][15]);   // beta @ W, from the spare operand row
                        p.Y[static_cast<size_t>(m) * p.N + n] = __float2bfloat16_rn(y);
                    }
                }
            }
            if (!whole) {
                asm volatile("bar.sync 1, 128;" ::: "memory");  // slot table / is_last reuse
                if (finish && warp == 2 && lane == 0) p.counters[tile] = 0u;
            }
            ++iter;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

struct Plan {
    int n_tiles, k_blocks, total_units, stages, stage_bytes, smem_bytes;
    size_t counters_bytes, total;
};
inline bool make_plan(int NW, bool norm, int K, int N, Plan* pl) {
    pl->n_tiles = (N + kBN - 1) / kBN;   // (the launcher may halve the tile width: counters are sized for that)
    pl->k_blocks = K / kBK;
    pl->total_units = pl->n_tiles * pl->k_blocks;
    pl->stage_bytes = NW * kWBytes + (norm ? 0 : kXBytes);
    const int xg = norm ? pl->k_blocks * kXBytes : 0;
    int stages = (kMaxSmem - 1024 - xg - kMiscBytes) / pl->stage_bytes;
    if (stages > 12) stages = 12;
    pl->stages = stages;
    pl->smem_bytes = 1024 + xg + stages * pl->stage_bytes + kMiscBytes;
    pl->counters_bytes = (static_cast<size_t>((N + 63) / 64) * 4 + 255) & ~size_t(255);
    pl->total = kDataOffset + static_cast<size_t>(kMaxGrid) * 2 * NW * kMaxM * kBN * 4;
    return stages >= 2;
}

template <int NW, int NORM>
ef_status launch(const void* X, const void* gamma, const void* beta, const void* W0, const void* W1, void* Y, int M, int K,
                 int N, float eps, void* ws, size_t ws_bytes, void* stream) {
    if (!X || !W0 || !Y || (NW == 2 && !W1) || (NORM && !gamma) || (NORM == 2 && !beta)) return EF_ERR_NULL;
    if (M <= 0 || K <= 0 || N <= 0) return EF_ERR_SHAPE;
    if (M > kMaxM || K % kBK != 0 || N % 8 != 0) return EF_ERR_UNSUPPORTED;
    if (NORM == 2 && M > kMaxM - 1) return EF_ERR_UNSUPPORTED;   // LayerNorm keeps one operand row for beta
    Plan pl;
    if (!make_plan(NW, NORM != 0, K, N, &pl)) return EF_ERR_UNSUPPORTED;  // NORM: X operand of the whole K must fit in shared memory
    if (static_cast<long long>(pl.n_tiles) * pl.k_blocks >= (1LL << 30)) return EF_ERR_UNSUPPORTED;
    if (kHeaderBytes + pl.counters_bytes > 65536) return EF_ERR_UNSUPPORTED;  // counters must lie in the init window
    if (!aligned(X, 16) || !aligned(W0, 16) || !aligned(Y, 16) || (NW == 2 && !aligned(W1, 16)) ||
        (NORM && !aligned(gamma, 16)) || (NORM == 2 && !aligned(beta, 16)))
        return EF_ERR_ALIGN;
    if (!ws || ws_bytes < pl.total) return EF_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return EF_ERR_ALIGN;
    DeviceInfo di;
    if (!current_device_info(&di)) return EF_ERR_CUDA;
    if (di.cc_major != 10) return EF_ERR_ARCH;

    CUtensorMap tmW0, tmW1, tmX;
    ef_status st;
    const uint64_t wdims[2] = {static_cast<uint64_t>(N), static_cast<uint64_t>(K)};
    const uint64_t wstrides[1] = {static_cast<uint64_t>(N) * 2};
    const uint32_t wbox[2] = {64, kBK};
    if ((st = encode_tmap_bf16(&tmW0, W0, 2, wdims, wstrides, wbox, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    if ((st = encode_tmap_bf16(&tmW1, NW == 2 ? W1 : W0, 2, wdims, wstrides, wbox, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    const uint64_t xdims[2] = {static_cast<uint64_t>(K), static_cast<uint64_t>(M)};
    const uint64_t xstrides[1] = {static_cast<uint64_t>(K) * 2};
    const uint32_t xbox[2] = {64, kMaxM};
    if ((st = encode_tmap_bf16(&tmX, X, 2, xdims, xstrides, xbox, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;

    static bool attr_set[64] = {};
    if (!attr_set[di.device]) {
        EF_CUDA_CHECK(cudaFuncSetAttribute(skinny_kernel<NW, NORM>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        attr_set[di.device] = true;
    }
    Params p;
    p.X = static_cast<const __nv_bfloat16*>(X);
    p.gamma = static_cast<const __nv_bfloat16*>(gamma);
    p.beta = static_cast<const __nv_bfloat16*>(beta);
    p.Y = static_cast<__nv_bfloat16*>(Y);
    p.M = M; p.K = K; p.N = N;
    p.lora = 0;
    p.pdl_mode = 0;
    p.out_scale = 1.f;
    p.n_tiles = pl.n_tiles; p.k_blocks = pl.k_blocks; p.total_units = pl.total_units;
    // Two k blocks per stage (weight boxes of 128 rows, 16 KiB: the copy engine moves more per request, and there are half as
    // many barrier round trips) whenever K allows it and at least two such stages fit; the partition then counts pairs.
    // Small calls (few k blocks per block): with 64-column tiles there are twice as many tiles, and when every block can
    // have a whole one (each streams its K x 64 slice of the weights, <= 384 KiB) no partial results are exchanged at all
    // (8x1024x4096: 64 blocks, 7.8 us against 8.4 us with 128-column tiles cut into four k ranges).
    int tile_n = kBN;
    {
        const int g0 = di.num_sms < kMaxGrid ? di.num_sms : kMaxGrid;
        const int n_tiles64 = (N + 63) / 64;
        if (pl.total_units / (g0 < pl.total_units ? g0 : pl.total_units) < 8 && n_tiles64 <= g0 &&
            static_cast<long long>(pl.k_blocks) * NW * kWAtomBytes <= 384 * 1024)
            tile_n = 64;
    }
    if (tile_n == 64) { pl.n_tiles = (N + 63) / 64; pl.total_units = pl.n_tiles * pl.k_blocks; p.n_tiles = pl.n_tiles; p.total_units = pl.total_units; }
    p.tile_n = tile_n;
    const bool pair = (pl.k_blocks % 2 == 0) && pl.stages >= 4;
    const int ku = pair ? 2 : 1;
    const int units = pl.total_units / ku, k_units = pl.k_blocks / ku;
    int grid = di.num_sms < units ? di.num_sms : units;
    if (grid > kMaxGrid) grid = kMaxGrid;
    if (tile_n == 64) {
        grid = pl.n_tiles;   // one block per whole 64-column tile
    } else if (pl.total_units / grid < 8) {
        // Few k blocks per block: the call is latency-bound, and ranges that straddle n-tile boundaries add partial
        // slots and arrivals.  Cut every n tile into the same number s of k ranges instead (s divides the k units)
        // as long as that keeps at least half of the blocks.
        int s = 0;
        for (int d = 1; d <= k_units; ++d)
            if (k_units % d == 0 && static_cast<long long>(pl.n_tiles) * d <= grid) s = d;
        if (s > 0 && pl.n_tiles * s * 2 >= grid) grid = pl.n_tiles * s;
    } else if (pl.n_tiles <= grid) {
        // Many k blocks per block and no more n tiles than SMs: one block per whole tile needs no partial slots, no arrival
        // counters and no merging block at the end of the kernel (measured: ~3.5 us), but leaves SMs idle.  A block alone
        // streams what it keeps in flight per ~2.9 us of memory latency (less with the larger boxes), so whole tiles win
        // when n_tiles such blocks already saturate HBM (gated MLP at 16x4096x11008: 86 blocks, 33.2 us against 38.2 us
        // with 148 split ranges; with the normalised X operand resident in shared memory there are fewer stages and the
        // split stays better).
        const double bytes = static_cast<double>(pl.total_units) * pl.stage_bytes;
        const double hbm = 5.7e6, per_block = static_cast<double>(pl.stages) * pl.stage_bytes / (pair ? 2.3 : 2.9);   // bytes per microsecond
        const double whole_rate = per_block * pl.n_tiles < hbm ? per_block * pl.n_tiles : hbm;
        if (bytes / whole_rate < bytes / hbm + 3.5) grid = pl.n_tiles;
    }
    if (pair) {
        const uint32_t wbox2[2] = {64, 2 * kBK};
        if ((st = encode_tmap_bf16(&tmW0, W0, 2, wdims, wstrides, wbox2, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
        if ((st = encode_tmap_bf16(&tmW1, NW == 2 ? W1 : W0, 2, wdims, wstrides, wbox2, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
        pl.stages /= 2;
    }
    p.pair = pair ? 1 : 0;
    p.base = (pl.total_units / (pair ? 2 : 1)) / grid;
    p.rem = (pl.total_units / (pair ? 2 : 1)) % grid;
    p.stages = pl.stages;
    p.eps = eps;
    uint8_t* w = static_cast<uint8_t*>(ws);
    p.status = reinterpret_cast<uint32_t*>(w);
    p.counters = reinterpret_cast<uint32_t*>(w + kHeaderBytes);
    p.partials = reinterpret_cast<float*>(w + kDataOffset);
    EF_CUDA_CHECK(launch_pdl(skinny_kernel<NW, NORM>, dim3(grid), dim3(kThreads), static_cast<size_t>(pl.smem_bytes),
                             static_cast<cudaStream_t>(stream), tmW0, tmW1, tmX, tmX, p));
    return EF_OK;
}

// The LoRA-fused linear for M <= 16 rows, both kernels on the weight-streaming kernel above:
//   launch_lora_head: T = alpha * X @ A   (A is a [K,16] weight: one n tile; few blocks, so few partials to merge)
//   launch_lora_tail: Y = [X | T] @ [W ; Bm], the rank-16 update as one extra k block.
size_t lora_tail_counters_bytes(int N) { return 256 + ((static_cast<size_t>((N + 63) / 64) * 4 + 255) & ~size_t(255)); }
constexpr int kLoraHeadGrid = 8;   // one n tile of 16 live columns, K / 64 k blocks: 8 blocks keep the ordered merge short
// partial slots of the head kernel (kLoraHeadGrid blocks) followed by those of the tail kernel: the two run concurrently
size_t lora_tail_partials_bytes() { return static_cast<size_t>(kLoraHeadGrid + kMaxGrid) * 2 * kMaxM * kBN * 4; }
static ef_status launch_plain(const void* X, const void* W, int w_rows, const void* T, const void* Bm, void* Y, int M, int K,
                              int N, float out_scale, int grid_cap, int pdl_mode, uint32_t* status, uint32_t* counters,
                              float* partials, const DeviceInfo& di, cudaStream_t stream) {
    const bool lora = T != nullptr;
    Plan pl;
    if (M > kMaxM || K % kBK != 0 || N % 8 != 0) return EF_ERR_UNSUPPORTED;
    // Two k blocks per stage when K / 64 is even (see launch()); the rank-16 update then takes a whole double stage.
    const bool pair = ((K / kBK) % 2 == 0);
    if (!make_plan(1, false, K + (lora ? (pair ? 2 : 1) * kBK : 0), N, &pl)) return EF_ERR_UNSUPPORTED;   // LoRA: one more stage than K needs
    if (static_cast<long long>(pl.n_tiles) * pl.k_blocks >= (1LL << 30)) return EF_ERR_UNSUPPORTED;
    CUtensorMap tmW, tmB, tmX, tmT;
    ef_status st;
    const uint64_t wdims[2] = {static_cast<uint64_t>(N), static_cast<uint64_t>(w_rows)};
    const uint64_t bdims[2] = {static_cast<uint64_t>(N), 16};
    const uint64_t wstrides[1] = {static_cast<uint64_t>(N) * 2};
    const uint32_t wbox[2] = {64, static_cast<uint32_t>(pair ? 2 * kBK : kBK)};
    if ((st = encode_tmap_bf16(&tmW, W, 2, wdims, wstrides, wbox, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    if ((st = encode_tmap_bf16(&tmB, lora ? Bm : W, 2, lora ? bdims : wdims, wstrides, wbox, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    const uint64_t xdims[2] = {static_cast<uint64_t>(K), static_cast<uint64_t>(M)};
    const uint64_t xstrides[1] = {static_cast<uint64_t>(K) * 2};
    const uint64_t tdims[2] = {16, static_cast<uint64_t>(M)};
    const uint64_t tstrides[1] = {16 * 2};
    const uint32_t xbox[2] = {64, kMaxM};
    if ((st = encode_tmap_bf16(&tmX, X, 2, xdims, xstrides, xbox, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    if ((st = encode_tmap_bf16(&tmT, lora ? T : X, 2, lora ? tdims : xdims, lora ? tstrides : xstrides, xbox, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    static bool attr_set[64] = {};
    if (!attr_set[di.device]) {
        EF_CUDA_CHECK(cudaFuncSetAttribute(skinny_kernel<1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        attr_set[di.device] = true;
    }
    Params p;
    p.X = static_cast<const __nv_bfloat16*>(X);
    p.gamma = nullptr;
    p.beta = nullptr;
    p.Y = static_cast<__nv_bfloat16*>(Y);
    p.M = M; p.K = K; p.N = N;
    p.lora = lora ? 1 : 0;
    p.tile_n = kBN;
    p.pair = pair ? 1 : 0;
    if (pair) pl.stages /= 2;
    p.pdl_mode = pdl_mode;
    p.out_scale = out_scale;
    // 64-column tiles when every block can then own a whole one (no partial exchange) and there are enough such blocks to
    // keep HBM busy (N = 8192: 128 blocks, 19.4 us against 24.5 us with split 128-column tiles; N = 4096: 64 blocks, no gain)
    const int n_tiles64 = (N + 63) / 64;
    const bool half = lora && n_tiles64 >= 76 && n_tiles64 <= di.num_sms && n_tiles64 <= grid_cap;
    if (half) { p.tile_n = 64; pl.n_tiles = n_tiles64; pl.total_units = pl.n_tiles * pl.k_blocks; }
    p.n_tiles = pl.n_tiles; p.k_blocks = pl.k_blocks; p.total_units = pl.total_units;
    const int units = pl.total_units / (pair ? 2 : 1);   // the partition counts pairs of k blocks when a stage holds two
    int grid = di.num_sms < units ? di.num_sms : units;
    if (grid > kMaxGrid) grid = kMaxGrid;
    if (grid > grid_cap) grid = grid_cap;
    if (half) grid = pl.n_tiles;
    p.base = units / grid;
    p.rem = units % grid;
    p.stages = pl.stages;
    p.eps = 0.f;
    p.status = status;
    p.counters = counters;
    p.partials = partials;
    EF_CUDA_CHECK(launch_pdl(skinny_kernel<1, 0>, dim3(grid), dim3(kThreads), static_cast<size_t>(pl.smem_bytes), stream, tmW,
                             tmB, tmX, tmT, p));
    return EF_OK;
}
ef_status launch_lora_head(const void* X, const void* A, void* T, int M, int K, float alpha, uint32_t* status,
                           uint32_t* counters, float* partials, const DeviceInfo& di, cudaStream_t stream) {
    // Waits for the kernel before it and only then lets the tail kernel start: the tail may then read X, W and Bm at once
    // and stream the weights while T is still being computed here.
    return launch_plain(X, A, K, nullptr, nullptr, T, M, K, 16, alpha, kLoraHeadGrid, 1, status, counters, partials, di, stream);
}
ef_status launch_lora_tail(const void* X, const void* W, const void* T, const void* Bm, void* Y, int M, int K, int N,
                           uint32_t* status, uint32_t* counters, float* partials, const DeviceInfo& di, cudaStream_t stream) {
    return launch_plain(X, W, K, T, Bm, Y, M, K, N, 1.f, kMaxGrid, 2, status, counters + 64,
                        partials + static_cast<size_t>(kLoraHeadGrid) * 2 * kMaxM * kBN, di, stream);
}

}  // namespace skinny
}  // namespace ef

extern "C" {

size_t ef_rmsnorm_matmul_workspace_bytes(int M, int K, int N) {
    ef::skinny::Plan pl;
    if (M <= 0 || K <= 0 || N <= 0 || K % ef::skinny::kBK != 0 || !ef::skinny::make_plan(1, true, K, N, &pl)) return 0;
    return pl.total;
}
ef_status ef_rmsnorm_matmul(const void* X, const void* gamma, const void* W, void* Y, int M, int K, int N, float eps,
                            void* ws, size_t ws_bytes, void* stream) {
    return ef::skinny::launch<1, 1>(X, gamma, nullptr, W, nullptr, Y, M, K, N, eps, ws, ws_bytes, stream);
}

size_t ef_rmsnorm_gated_mlp_workspace_bytes(int M, int K, int N) {
    ef::skinny::Plan pl;
    if (M <= 0 || K <= 0 || N <= 0 || K % ef::skinny::kBK != 0 || !ef::skinny::make_plan(2, true, K, N, &pl)) return 0;
    return pl.total;
}
ef_status ef_rmsnorm_gated_mlp(const void* X, const void* gamma, const void* Wgate, const void* Wup, void* Y, int M, int K,
                               int N, float eps, void* ws, size_t ws_bytes, void* stream) {
    // Up to 8 rows go through in one launch with the hi/lo operand split (the spare operand rows carry the rounding remainder
    // of x*gamma).  More rows have no spare operand rows, and the plain bf16 operand is not accurate enough for the gated
    // product (a small SiLU(g) times a large u: single elements miss 1e-2 + 1e-2*|ref| by up to 3x), so 9..16 rows run as two
    // launches of <= 8 rows each on the same workspace: twice the weight traffic, the same accuracy as for M <= 8.
    if (M > 8 && M <= ef::skinny::kMaxM && X && Y && K > 0 && N > 0) {
        const ef_status st = ef::skinny::launch<2, 1>(X, gamma, nullptr, Wgate, Wup, Y, 8, K, N, eps, ws, ws_bytes, stream);
        if (st != EF_OK) return st;
        return ef::skinny::launch<2, 1>(static_cast<const __nv_bfloat16*>(X) + static_cast<size_t>(8) * K, gamma, nullptr, Wgate,
                                        Wup, static_cast<__nv_bfloat16*>(Y) + static_cast<size_t>(8) * N, M - 8, K, N, eps, ws,
                                        ws_bytes, stream);
    }
    return ef::skinny::launch<2, 1>(X, gamma, nullptr, Wgate, Wup, Y, M, K, N, eps, ws, ws_bytes, stream);
}

size_t ef_layernorm_matmul_workspace_bytes(int M, int K, int N) {
    ef::skinny::Plan pl;
    if (M <= 0 || K <= 0 || N <= 0 || K % ef::skinny::kBK != 0 || !ef::skinny::make_plan(1, true, K, N, &pl)) return 0;
    return pl.total;
}
ef_status ef_layernorm_matmul(const void* X, const void* gamma, const void* beta, const void* W, void* Y, int M, int K,
                              int N, float eps, void* ws, size_t ws_bytes, void* stream) {
    return ef::skinny::launch<1, 2>(X, gamma, beta, W, nullptr, Y, M, K, N, eps, ws, ws_bytes, stream);
}

size_t ef_gated_mlp_workspace_bytes(int M, int K, int N) {
    ef::skinny::Plan pl;
    if (M <= 0 || K <= 0 || N <= 0 || K % ef::skinny::kBK != 0 || !ef::skinny::make_plan(2, false, K, N, &pl)) return 0;
    return pl.total;
}
ef_status ef_gated_mlp(const void* X, const void* Wgate, const void* Wup, void* Y, int M, int K, int N, void* ws,
                       size_t ws_bytes, void* stream) {
    return ef::skinny::launch<2, 0>(X, nullptr, nullptr, Wgate, Wup, Y, M, K, N, 0.f, ws, ws_bytes, stream);
}

}  // extern "C"
