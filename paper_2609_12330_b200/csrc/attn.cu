// ef_qknorm_attn: (causal) prefill attention with RMS-normalised queries and keys.
//
// Algebra (Table 1, factor motion; Section 7.3, QK-normalized MLA): with rq_i, rk_j the inverse
// RMS of query row i / key row j,
//     s_ij = scale * sum_d (rq_i q_id gq_d gk_d) (rk_j k_jd) ,
// so the gamma product and rq_i are folded into the Q tile once per block (rewritten in shared
// memory as fp16), scale * log2(e) is folded into the exp2 FMA on the logits, and the key factor is applied
// once per key by a pre-pass kernel that writes Khat = fp16(k * rk) (read back from L2 by the main
// kernel; |Khat_d| <= sqrt(128), so fp16's 11-bit mantissa is safe and four times finer than bf16;
// for the same reason P, which lies in [0, 2^8], is handed to the PV MMA as fp16).  The key factor is NOT applied on the logits inside the block: that needs one
// shared-memory read per four logits, and shared-memory reads of ordinary warps starve while the
// tensor core streams Q and K tiles (a 128x128x16 MMA with both operands in shared memory uses the
// full 128 B/clk; measured: an LDS.128 then takes ~600 cycles).  The softmax loop therefore touches
// no shared memory at all.
//
// Execution form (Figure 4, M2): work items (batch*head, pair of 128-row Q tiles) = axis m, pulled
// heaviest-first from a global counter by one persistent block per SM (the next item's Q tiles
// are fetched while the current item drains); loop
// over 128-key K/V tiles = axis p, rolling state <max, sum, value> with the repair
// h(c,s,s') = c * exp(s - s').  The repair is applied lazily: the accumulated value is rescaled
// only when the running maximum grows by more than 2^8 (any reference maximum is exact in real
// arithmetic because numerator and normaliser use the same one).  Because Q and K are normalised
// the logits are bounded a priori (128 * max|gq gk| * scale); when that bound is at most 2^40 in
// exp2 units it IS the reference: no maximum is computed and no repair is ever needed.  Causal:
// tiles above the diagonal are never visited, only the diagonal tile is masked.
//
// Pipeline per block (320 threads): warp 0 = TMA producer (Q once, K/V rings), warp 1 = single
// thread issuing tcgen05.mma (S_t = Q_t Khat^T into TMEM, O_t += P_t V with P read from TMEM),
// warps 2..5 / 6..9 = softmax groups for Q tile 0 / 1 (one thread per row: tcgen05.ld S, packed
// fp32x2 FMA + exp2, write P as bf16 back into the S columns, rescale O when needed, final
// O / l).  While one group runs its softmax the tensor core works on the other tile.  Score and
// probability matrices never leave the SM (Section 7.2).
#include "host.cuh"
#include "ptx.cuh"

namespace ef {
namespace attn {

constexpr int kD = 128;
constexpr int kT = 128;                           // tile edge (queries and keys)
constexpr int kHalfBytes = kT * 128;              // [128 rows][64 d] bf16, 128B swizzle
constexpr int kTileBytes = 2 * kHalfBytes;        // 32 KiB
constexpr int kKVSlots = 4;                        // K/V tiles in shared memory: two double slots {V_j, K_j+1}
constexpr int kThreads = 320;
constexpr int kKeyRowsPerThread = 4;               // pre-pass: key rows per thread
constexpr uint32_t kTmemCols = 512;               // S0 | S1 | O0 | O1, 128 fp32 columns each
// shared memory map (offsets from the 1024-aligned base)
constexpr int kOffQ = 0;                                          // 2 tiles
constexpr int kOffKV = kOffQ + 2 * kTileBytes;                    // kKVSlots tiles
constexpr int kOffGamma = kOffKV + kKVSlots * kTileBytes;         // [128 floats] gq*gk
constexpr int kOffBars = kOffGamma + kD * 4;
constexpr int kSmemBytes = 1024 + kOffBars + 512;
constexpr int kWorkCounterWord = 16;               // uint32 index into the workspace header
constexpr int kDoneCounterWord = 17;
constexpr float kRescaleThreshold = 8.0f;         // log2 units
constexpr float kFixedRefLimit = 40.0f;           // log2 units: use the a-priori logit bound as softmax reference

struct Params {
    const __nv_bfloat16* gamma_q;
    const __nv_bfloat16* gamma_k;
    __nv_bfloat16* O;     // [BH][S][128]
    int BH, S, nq, n_pairs, causal;
    int Hq, Hkv;          // BH = B * Hq query heads; K and V have B * Hkv heads (consecutive query heads share one)
    int window, sinks;    // causal only: key j is visible to query i iff j <= i and (j > i - window or j < sinks); 0 = no window
    float eps, scale_log2;
    int total_items;
    int o_vec8;           // O is 32-byte aligned: the epilogue may use 256-bit stores
    uint32_t* status;
    uint32_t* header;   // workspace header: work counter / done counter for the persistent grid
};

__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status, uint32_t site) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, status, site)) != 0;
}
// Packed fp32x2 arithmetic (sm_100): one instruction works on two adjacent logits.
__device__ __forceinline__ uint64_t pack_f32x2(uint32_t lo, uint32_t hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ void st_global_v8(void* dst, const uint32_t* v) {   // 32-byte aligned destination
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(v[0]), "r"(v[1]), "r"(v[2]),
                 "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// ---------------------------------------------------------------------------------------------
// pre-pass: Khat[row][d] = fp16(K[row][d] * rsqrt(mean_d K[row][d]^2 + eps) * gq[d] * gk[d]): both gammas ride
// on the keys (the logit only needs their product), so the query side needs no per-column factor.  16 threads
// per key row, one 16-byte piece each, so every load of the grid is in flight at once.  |k * rk| <= sqrt(128);
// the clamp only matters for huge gammas.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) key_normalize_kernel(const __nv_bfloat16* __restrict__ K,
                                                            const __nv_bfloat16* __restrict__ gamma_q,
                                                            const __nv_bfloat16* __restrict__ gamma_k,
                                                            __nv_bfloat16* __restrict__ Khat, long long rows, float eps) {
    pdl_launch_dependents();
    pdl_wait();
    const int sub = threadIdx.x & 15;
    float g[8];   // gq*gk of this thread's 8 columns (2-byte loads: the gammas need no 16-byte alignment)
#pragma unroll
    for (int i = 0; i < 8; ++i) g[i] = __bfloat162float(gamma_q[sub * 8 + i]) * __bfloat162float(gamma_k[sub * 8 + i]);
    // kKeyRowsPerThread rows per thread, 16 rows apart: all of a thread's loads are issued before the first use
    const long long row0 = static_cast<long long>(blockIdx.x) * (16 * kKeyRowsPerThread) + (threadIdx.x >> 4);
    uint4 v[kKeyRowsPerThread];
#pragma unroll
    for (int u = 0; u < kKeyRowsPerThread; ++u) {
        const long long row = row0 + 16 * u;
        v[u] = make_uint4(0u, 0u, 0u, 0u);
        if (row < rows) v[u] = __ldg(reinterpret_cast<const uint4*>(K + row * kD) + sub);
    }
#pragma unroll
    for (int u = 0; u < kKeyRowsPerThread; ++u) {
        const long long row = row0 + 16 * u;
        const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
        float lo[4], hi[4], ss = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            lo[i] = __uint_as_float(w[i] << 16);
            hi[i] = __uint_as_float(w[i] & 0xFFFF0000u);
            ss += lo[i] * lo[i] + hi[i] * hi[i];
        }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        const float rk = rsqrtf(ss * (1.f / kD) + eps);
        if (row < rows) {
            uint32_t o4[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                o4[i] = pack_f16x2(fminf(fmaxf(lo[i] * rk * g[2 * i], -65504.f), 65504.f), fminf(fmaxf(hi[i] * rk * g[2 * i + 1], -65504.f), 65504.f));
            reinterpret_cast<uint4*>(Khat + row * kD)[sub] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// main kernel (persistent: one block per SM pulls work items from a global counter)
// ---------------------------------------------------------------------------------------------
// Work item = (batch*head, pair of Q tiles); item index order is heaviest pair first, so greedy
// pulling is longest-processing-time-first scheduling.
// A pair visits a LIST of key tiles, shared by its two Q tiles: the tiles of the (causal, windowed) range of either
// tile, preceded by key tile 0 when attention sinks are in use and the window has moved past it.  Entry a of the
// list is key tile kt(a); Q tile t takes part in entry a iff part(t, a).
struct Item {
    int bh, qt0;
    int n_kv;        // entries of the list
    int lo;          // first key tile of the window range
    int sink;        // 1: entry 0 is key tile 0, visited for the sink keys only
    int wf0, wl0, wf1, wl1;   // first and last entry of tile t's window range (wl < wf: the tile is absent)
    __device__ __forceinline__ int wf(int t) const { return t ? wf1 : wf0; }
    __device__ __forceinline__ int wl(int t) const { return t ? wl1 : wl0; }
    __device__ __forceinline__ int kt(int a) const { return sink ? (a == 0 ? 0 : lo + a - 1) : lo + a; }
    __device__ __forceinline__ bool present(int t) const { return wl(t) >= wf(t); }
    __device__ __forceinline__ bool part(int t, int a) const { return (sink && a == 0 && present(t)) || (a >= wf(t) && a <= wl(t)); }
    __device__ __forceinline__ int first(int t) const { return (sink && present(t)) ? 0 : wf(t); }
    __device__ __forceinline__ int last(int t) const { return wl(t); }
};
// geometry of the pair whose first Q tile is qt0 (no division: the consumers' per-item path).  WIN = false is the
// kernel instance without a sliding window: the list is key tiles 0..hi, every field below folds to a constant
// and part(t, a) is a single comparison again.
template <bool WIN>
__device__ __forceinline__ Item item_from(const Params& p, int bh, int qt0) {
    Item g;
    g.bh = bh;
    g.qt0 = qt0;
    if constexpr (!WIN) {
        const bool has_q1 = qt0 + 1 < p.nq;
        const int hi0 = p.causal ? qt0 : p.nq - 1;
        const int hi1 = has_q1 ? (p.causal ? qt0 + 1 : p.nq - 1) : -1;
        g.lo = 0; g.sink = 0;
        g.n_kv = max(hi0, hi1) + 1;
        g.wf0 = 0; g.wl0 = hi0;
        g.wf1 = 0; g.wl1 = hi1;
        return g;
    } else {
    int lo_t[2], hi_t[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int qt = qt0 + t;
        hi_t[t] = p.causal ? qt : p.nq - 1;
        const int jmin = p.window > 0 ? max(0, qt * kT - p.window + 1) : 0;   // lowest key any row of the tile sees
        lo_t[t] = jmin / kT;
        if (qt >= p.nq) hi_t[t] = lo_t[t] - 1;                                 // absent tile
    }
    g.lo = lo_t[0];
    g.sink = (p.sinks > 0 && g.lo > 0) ? 1 : 0;
    const int hi = max(hi_t[0], hi_t[1]);
    g.n_kv = hi - g.lo + 1 + g.sink;
    g.wf0 = lo_t[0] - g.lo + g.sink; g.wl0 = hi_t[0] - g.lo + g.sink;
    g.wf1 = lo_t[1] - g.lo + g.sink; g.wl1 = hi_t[1] - g.lo + g.sink;
    // key tile 0 is inside the list but below a tile's window: it still holds that tile's sink keys
    if (!g.sink && p.sinks > 0 && g.lo == 0) {
        if (g.wl0 >= g.wf0) g.wf0 = 0;
        if (g.wl1 >= g.wf1) g.wf1 = 0;
    }
    return g;
    }
}
template <bool WIN>
__device__ __forceinline__ Item item_geom(const Params& p, int item) {
    const int pair = p.n_pairs - 1 - item / p.BH;
    return item_from<WIN>(p, item - (item / p.BH) * p.BH, 2 * pair);
}

template <bool WIN>
__global__ void __launch_bounds__(kThreads, 1)
qknorm_attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    float* gprod = reinterpret_cast<float*>(smem + kOffGamma);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kOffBars);
    uint64_t* q_full = bars;                 // [2]  TMA -> softmax group t (raw Q tile t of the item landed)
    uint64_t* q_empty = bars + 2;            // [2]  MMA -> TMA (last QK^T of tile t done: Q tile t may be overwritten)
    uint64_t* q_ready = bars + 4;            // [2]  softmax group t -> MMA (Q tile t rewritten)
    uint64_t* kv_full = bars + 6;            // [2]  K/V ring of two double slots: pair number n lives in double slot n & 1,
    uint64_t* kv_empty = bars + 11;          // [2]        phase (n >> 1) & 1
    uint64_t* s_full = bars + 16;            // [2]  MMA -> softmax group t
    uint64_t* p_full = bars + 18;            // [2]  softmax group t -> MMA
    uint64_t* o_done = bars + 20;            // [2]  MMA -> softmax group t (PV finished)
    uint64_t* o_free = bars + 22;            // [2]  softmax group t -> MMA (O_t read out: may be overwritten)
    uint64_t* item_full = bars + 24;         // [2]  TMA -> everyone (work item published)
    uint64_t* item_empty = bars + 26;        // [2]  everyone -> TMA (item slot read)
    int2* item_ring = reinterpret_cast<int2*>(bars + 28);   // [2]  {batch*head, first Q tile}; x < 0: no more work
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 30);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int t = 0; t < 2; ++t) {
            mbar_init(&q_full[t], 1); mbar_init(&q_empty[t], 1);
            mbar_init(&q_ready[t], 4);
            mbar_init(&s_full[t], 1); mbar_init(&p_full[t], 4); mbar_init(&o_done[t], 1); mbar_init(&o_free[t], 4);
            mbar_init(&item_full[t], 1); mbar_init(&item_empty[t], 9);   // MMA thread + 8 softmax warps
        }
        for (int i = 0; i < kKVSlots; ++i) { mbar_init(&kv_full[i], 1); mbar_init(&kv_empty[i], 1); }
        *abort_flag = 0u;
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
    pdl_launch_dependents();
    pdl_wait();  // Khat (previous kernel), gammas, O of earlier calls: no global access above this line
    if (threadIdx.x >= 64 && threadIdx.x < 64 + kD) {
        const int d = threadIdx.x - 64;
        gprod[d] = __bfloat162float(p.gamma_q[d]) * __bfloat162float(p.gamma_k[d]);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------ TMA producer + work fetch ------------------------------
        if (lane == 0) {
            tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
            uint32_t pc = 0;   // K/V pairs loaded so far: pair = {V of one list entry, K of the next} in one double slot, ONE barrier
            uint32_t n_items = 0;
            uint32_t item = atomicAdd(&p.header[kWorkCounterWord], 1u);
            bool ok = true;
            while (ok) {
                const int slot = n_items & 1;
                if (!mbar_wait(&item_empty[slot], ((n_items >> 1) & 1) ^ 1u, abort_flag, p.status, 1)) break;
                const bool valid = item < static_cast<uint32_t>(p.total_items);
                const Item g = item_geom<WIN>(p, valid ? static_cast<int>(item) : 0);
                item_ring[slot] = valid ? make_int2(g.bh, g.qt0) : make_int2(-1, 0);
                mbar_arrive(&item_full[slot]);
                if (!valid) break;
                const uint32_t next = atomicAdd(&p.header[kWorkCounterWord], 1u);   // latency hides behind the copies
                // Q tile t of the new item goes in as soon as the previous item's last QK^T of tile t is done
                // (tile 0 finishes one key tile earlier than tile 1 under the causal mask), so the load is
                // hidden behind the previous item's tail.  Order: Q0, K(0), Q1, V(0), then the remaining K/V.
                auto load_q = [&](int t) -> bool {
                    if (n_items > 0 && !mbar_wait(&q_empty[t], (n_items - 1) & 1, abort_flag, p.status, 2)) return false;
                    mbar_expect_tx(&q_full[t], kTileBytes);   // rows beyond S are out of bounds -> zero fill
                    tma_load_3d(smem + kOffQ + t * kTileBytes, &tmQ, &q_full[t], 0, (g.qt0 + t) * kT, g.bh);
                    tma_load_3d(smem + kOffQ + t * kTileBytes + kHalfBytes, &tmQ, &q_full[t], 64, (g.qt0 + t) * kT, g.bh);
                    return true;
                };
                if (!load_q(0)) break;
                const int kvz = (p.Hq == p.Hkv) ? g.bh : (g.bh / p.Hq) * p.Hkv + (g.bh % p.Hq) / (p.Hq / p.Hkv);   // K/V head
                // The K/V ring holds two double slots.  A double slot carries what one step of the MMA issuer consumes -- V of
                // list entry a and K of entry a+1 -- under ONE full/empty barrier pair (the issuer spends its time on barrier
                // round trips, so there are as few as possible); the item's first K tile travels alone in a double slot.
                auto load_pair = [&](int a_v, int a_k) -> bool {   // a_v < 0: no V; a_k < 0: no K
                    const uint32_t d = pc & 1u;
                    if (!mbar_wait(&kv_empty[d], ((pc >> 1) & 1) ^ 1u, abort_flag, p.status, 3)) return false;
                    uint8_t* base = smem + kOffKV + d * 2 * kTileBytes;
                    mbar_expect_tx(&kv_full[d], ((a_v >= 0) + (a_k >= 0)) * kTileBytes);
                    if (a_v >= 0) {
                        const int j = g.kt(a_v);
                        tma_load_3d(base, &tmV, &kv_full[d], 0, j * kT, kvz);
                        tma_load_3d(base + kHalfBytes, &tmV, &kv_full[d], 64, j * kT, kvz);
                    }
                    if (a_k >= 0) {
                        const int j = g.kt(a_k);
                        tma_load_3d(base + kTileBytes, &tmK, &kv_full[d], 0, j * kT, kvz);
                        tma_load_3d(base + kTileBytes + kHalfBytes, &tmK, &kv_full[d], 64, j * kT, kvz);
                    }
                    ++pc;
                    return true;
                };
                ok = load_pair(-1, 0) && load_q(1);
                for (int a = 0; a < g.n_kv && ok; ++a) ok = load_pair(a, a + 1 < g.n_kv ? a + 1 : -1);
                if (!ok) break;
                item = next;
                ++n_items;
            }
            // The block that stops fetching last re-arms the work counter for the next call.
            __threadfence();
            const uint32_t prev = atomicAdd(&p.header[kDoneCounterWord], 1u);
            if (prev == gridDim.x - 1) {
                p.header[kWorkCounterWord] = 0u;
                p.header[kDoneCounterWord] = 0u;
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            constexpr uint32_t idesc_qk = make_idesc_f16(kT, kT, 0, 0, 0, 0);  // A = Qhat fp16 (K-major), B = Khat fp16 (K-major)
            constexpr uint32_t idesc_pv = make_idesc_f16(kT, kD, 0, 1, 1, 1);  // A = P bf16 (TMEM),   B = V bf16 (MN-major)
            const uint32_t sQ = smem_u32(smem + kOffQ), sKV = smem_u32(smem + kOffKV);
            // descriptor words: hi is constant per operand kind, lo = base + compile-time offset
            constexpr uint32_t hi_kmajor = smem_desc_hi(1024, kSwizzle128B);   // Q and K tiles
            constexpr uint32_t hi_v = smem_desc_hi(1024, kSwizzle128B);        // V tile (MN-major: LBO in lo word)
            const uint32_t q_lo[2] = {smem_desc_lo(sQ, 16), smem_desc_lo(sQ + kTileBytes, 16)};
            auto issue_qk = [&](int t, uint32_t kaddr) {
                const uint32_t a0 = q_lo[t], b0 = smem_desc_lo(kaddr, 16), d = tmem_base + t * kT;
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk) {
                    const uint32_t off = ((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4;
                    umma_ss_w(d, a0 + off, hi_kmajor, b0 + off, hi_kmajor, idesc_qk, kk != 0 ? 1u : 0u);
                }
            };
            auto issue_pv = [&](int t, uint32_t vaddr, uint32_t accumulate) {
                const uint32_t b0 = smem_desc_lo(vaddr, kHalfBytes), d = tmem_base + 2 * kT + t * kD, a = tmem_base + t * kT;
#pragma unroll
                for (int kk = 0; kk < kT / 16; ++kk)
                    umma_ts_w(d, a + kk * 8, b0 + kk * (2048 >> 4), hi_v, idesc_pv, kk != 0 ? 1u : accumulate);
            };
            uint32_t pu = 0;              // K/V pairs (double slots) consumed so far
            // with the a-priori logit bound nobody waits for a PV but the epilogue: one commit per item and tile suffices
            float gmax_i = 0.f;
            for (int d = 0; d < kD; ++d) gmax_i = fmaxf(gmax_i, fabsf(gprod[d]));
            const bool every_pv = !(static_cast<float>(kD) * gmax_i * p.scale_log2 <= kFixedRefLimit);
            uint32_t n_items = 0;
            uint32_t cp[2] = {0u, 0u};    // p_full completions consumed per tile
            bool ok = true;
            while (ok) {
                const int slot = n_items & 1;
                if (!mbar_wait(&item_full[slot], (n_items >> 1) & 1, abort_flag, p.status, 4)) break;
                const int2 item = item_ring[slot];
                mbar_arrive(&item_empty[slot]);
                if (item.x < 0) break;
                const Item g = item_from<WIN>(p, item.x, item.y);
                // Entry a of the item's key list: tile t takes part iff g.part(t, a).  QK^T of entry a+1 is always
                // issued during step a (right after the tile's PV of entry a, if it has one), so the K/V ring is
                // released in list order whatever subset of entries a tile visits.
                {
                    const uint32_t st0 = pu & 1u;   // double slot of the item's first K tile
                    const uint32_t k0addr = sKV + st0 * 2 * kTileBytes + kTileBytes;
                    bool k_waited = false;
                    for (int t = 0; t < 2 && ok; ++t) {
                        ok = mbar_wait(&q_ready[t], n_items & 1, abort_flag, p.status, 4);
                        if (ok && n_items > 0) ok = mbar_wait(&o_free[t], (n_items - 1) & 1, abort_flag, p.status, 4);
                        if (!ok) break;
                        if (g.part(t, 0)) {
                            if (!k_waited) {
                                if (!mbar_wait(&kv_full[st0], (pu >> 1) & 1, abort_flag, p.status, 5)) { ok = false; break; }
                                k_waited = true;
                            }
                            tc_fence_after();
                            issue_qk(t, k0addr);
                            umma_commit(&s_full[t]);
                        }
                        // tile t's last QK^T (or none at all): its Q tile may be overwritten
                        if (!g.present(t) || g.last(t) == 0) umma_commit(&q_empty[t]);
                    }
                    if (!ok) break;
                    umma_commit(&kv_empty[st0]);
                    ++pu;
                }
                for (int j = 0; j < g.n_kv && ok; ++j, ++pu) {
                    const uint32_t st = pu & 1u;   // double slot of this step: V of entry j, K of entry j+1
                    const uint32_t vaddr = sKV + st * 2 * kTileBytes, kaddr = vaddr + kTileBytes;
                    // The tiles of this step landed long ago: look at their barrier now, while the softmax groups are still
                    // busy, so that nothing but the MMAs follows a group's hand-over on the critical path.
                    if (!mbar_wait(&kv_full[st], (pu >> 1) & 1, abort_flag, p.status, 7)) { ok = false; break; }
                    tc_fence_after();
                    for (int t = 0; t < 2 && ok; ++t) {
                        if (g.part(t, j)) {
                            if (!mbar_wait(&p_full[t], cp[t] & 1, abort_flag, p.status, 6)) { ok = false; break; }
                            ++cp[t];
                            tc_fence_after();
                            issue_pv(t, vaddr, j > g.first(t) ? 1u : 0u);
                            if (every_pv || j == g.last(t)) umma_commit(&o_done[t]);
                        }
                        if (j + 1 < g.n_kv && g.part(t, j + 1)) {
                            issue_qk(t, kaddr);
                            umma_commit(&s_full[t]);
                            if (j + 1 == g.last(t)) umma_commit(&q_empty[t]);   // tile t's last QK^T: its Q tile is free
                        }
                    }
                    if (!ok) break;
                    umma_commit(&kv_empty[st]);   // all MMAs that read this double slot are issued
                }
                if (!ok) break;
                ++n_items;
            }
        }
    } else {
        // ------------------------------ softmax groups ------------------------------
        const int t = (warp - 2) >> 2;             // 0: Q tile 0, 1: Q tile 1
        const int q = warp & 3;                    // TMEM lane quadrant
        const int r = q * 32 + lane;               // row within the tile
        const uint32_t lane_sel = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t tS = tmem_base + t * kT + lane_sel;
        const uint32_t tO = tmem_base + 2 * kT + t * kD + lane_sel;
        // Normalised queries and keys bound every logit: |qhat . khat| <= 128 * max_d |gq_d gk_d|
        // (Cauchy-Schwarz on rows of RMS <= 1).  When that bound is modest the softmax needs no running
        // maximum at all: exp2(x - bound) can neither overflow nor lose the row (p >= 2^(-2*bound)),
        // and numerator and normaliser share the reference, so the result is exact in real arithmetic.
        float gmax = 0.f;
#pragma unroll 8
        for (int d = 0; d < kD; ++d) gmax = fmaxf(gmax, fabsf(gprod[d]));
        const float bound = static_cast<float>(kD) * gmax * p.scale_log2;
        const bool fixed_ref = bound <= kFixedRefLimit;
        const float rq = p.scale_log2;   // the logits' only remaining factor: scale * log2(e), the same for every row
        const uint64_t rq2 = pack_f32x2(__float_as_uint(rq), __float_as_uint(rq));
        uint32_t n_items = 0;
        uint32_t cs = 0;   // s_full completions consumed by this group
        uint32_t co = 0;   // PV (o_done) completions of earlier items of this group's tile
        bool ok = true;
        while (ok) {
            const int slot = n_items & 1;
            if (!warp_wait(&item_full[slot], (n_items >> 1) & 1, abort_flag, p.status, 9)) break;
            const int2 item = item_ring[slot];
            __syncwarp();
            if (lane == 0) mbar_arrive(&item_empty[slot]);
            if (item.x < 0) break;
            const Item g = item_from<WIN>(p, item.x, item.y);
            const bool present = g.present(t);
            const int my_count = present ? g.wl(t) - g.wf(t) + 1 + g.sink : 0;   // list entries this tile takes part in
            const int my_commits = fixed_ref ? (my_count > 0 ? 1 : 0) : my_count;      // o_done completions of this item
            const int qt = g.qt0 + t;
            const int row_g = qt * kT + r;             // query index within the sequence
            if (!warp_wait(&q_full[t], n_items & 1, abort_flag, p.status, 9)) break;
            if (present) {
                // in-place rewrite of this thread's query row: qhat_d = fp16(q_d * rq_i); |q * rq| <= sqrt(128)
                // whatever the scale of q, so fp16 is safe (the gammas ride on the keys)
                uint8_t* qrow = smem + kOffQ + t * kTileBytes + r * 128;
                uint4 v[16];   // the whole row stays in registers between the two passes
                float ss4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    v[c] = *reinterpret_cast<const uint4*>(qrow + (c >> 3) * kHalfBytes + (((c & 7) ^ (r & 7)) << 4));
                    const uint32_t w[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float a = __uint_as_float(w[i] << 16), b = __uint_as_float(w[i] & 0xFFFF0000u);
                        ss4[i] = fmaf(a, a, fmaf(b, b, ss4[i]));
                    }
                }
                const float rqi = rsqrtf(((ss4[0] + ss4[1]) + (ss4[2] + ss4[3])) * (1.f / kD) + p.eps);
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const uint32_t w[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
                    uint32_t o4[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        o4[i] = pack_f16x2(__uint_as_float(w[i] << 16) * rqi, __uint_as_float(w[i] & 0xFFFF0000u) * rqi);
                    *reinterpret_cast<uint4*>(qrow + (c >> 3) * kHalfBytes + (((c & 7) ^ (r & 7)) << 4)) = make_uint4(o4[0], o4[1], o4[2], o4[3]);
                }
                fence_proxy_async_smem();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&q_ready[t]);   // every warp, every item (also when this tile has no work)
            float m_ref = fixed_ref ? bound : -INFINITY, l_sum = 0.f;
            int np = 0;   // entries processed so far
            for (int a = g.first(t); a <= g.last(t) && ok; ++a) {
                if (WIN && !g.part(t, a)) continue;
                const int j = g.kt(a);   // key tile of this entry
                if (!warp_wait(&s_full[t], cs & 1, abort_flag, p.status, 10)) { ok = false; break; }
                ++cs;
                tc_fence_after();
                uint32_t s[4][32];
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, s[c]);
                tmem_wait_ld();
                // Masked tiles only: the diagonal tile, the ragged last key tile, and under a sliding window the
                // tiles that reach below some row's window (the sink tile among them: only its sink keys count).
                const bool diag = p.causal && (j == qt);
                if constexpr (!WIN) {
                    if (diag || (j * kT + kT > p.S)) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                const int col = c * 32 + i;
                                if (!((!diag || col <= r) && (j * kT + col < p.S))) s[c][i] = 0xFF800000u;  // -inf
                            }
                        }
                    }
                } else {
                    const bool below = j * kT <= qt * kT + kT - 1 - p.window;
                    if (diag || below || (j * kT + kT > p.S)) {
                        // column c of this tile is visible to this row iff c <= hi and (c >= lo or c < sk)
                        const int hi = min(diag ? r : kT - 1, p.S - 1 - j * kT);
                        const int lo = qt * kT + r - p.window + 1 - j * kT;
                        const int sk = p.sinks - j * kT;
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                const int col = c * 32 + i;
                                if (!(col <= hi && (col >= lo || col < sk))) s[c][i] = 0xFF800000u;  // -inf
                            }
                        }
                    }
                }
                // Running maximum with lazy repair -- skipped entirely when the logits are bounded a priori.
                float o_scale = 1.f;
                bool need = false;
                if (!fixed_ref) {
                    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
#pragma unroll
                        for (int i = 0; i < 32; i += 2)
                            mx[(i >> 1) & 3] = max3(mx[(i >> 1) & 3], __uint_as_float(s[c][i]), __uint_as_float(s[c][i + 1]));
                    }
                    const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * rq;   // rq = scale * log2(e) > 0
                    need = m_tile > m_ref + kRescaleThreshold;
                    if (need) {
                        o_scale = fast_exp2(m_ref - m_tile);  // 0 on the first tile (m_ref = -inf)
                        l_sum *= o_scale;
                        m_ref = m_tile;
                    }
                }
                // p = exp2(acc * scale*log2e - m_ref): packed FMA, two exp2, packed row sum (4 independent accumulators)
                const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;   // a row may see nothing in its first tiles
                const uint64_t nm2 = pack_f32x2(__float_as_uint(-m_use), __float_as_uint(-m_use));
                uint64_t acc2[4] = {0ull, 0ull, 0ull, 0ull};
                uint32_t pk[64];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        float a, b;
                        unpack_f32x2(fma_f32x2(pack_f32x2(s[c][2 * i], s[c][2 * i + 1]), rq2, nm2), a, b);
                        const float p0 = fast_exp2(a), p1 = fast_exp2(b);
                        acc2[i & 3] = add_f32x2(acc2[i & 3], pack_f32x2(__float_as_uint(p0), __float_as_uint(p1)));
                        pk[c * 16 + i] = pack_bf16x2(p0, p1);
                    }
                }
                {
                    float a, b;
                    unpack_f32x2(add_f32x2(add_f32x2(acc2[0], acc2[1]), add_f32x2(acc2[2], acc2[3])), a, b);
                    l_sum += a + b;
                }
                // P (bf16) overwrites the first 64 columns of this thread's own S row
                {
                    uint32_t (&lo)[32] = *reinterpret_cast<uint32_t (*)[32]>(&pk[0]);
                    uint32_t (&hi)[32] = *reinterpret_cast<uint32_t (*)[32]>(&pk[32]);
                    tmem_st32(tS, lo);
                    tmem_st32(tS + 32, hi);
                }
                // rescale the accumulated value when some row of this warp moved its reference maximum
                if (np > 0 && __any_sync(0xffffffffu, need)) {
                    if (!warp_wait(&o_done[t], (co + np - 1) & 1, abort_flag, p.status, 12)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t ov[32];
                        tmem_ld32(tO + c * 32, ov);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * o_scale);
                        tmem_st32(tO + c * 32, ov);
                    }
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_full[t]);
                ++np;
            }
            if (!ok) break;
            // epilogue: read O out of TMEM (then the next item may overwrite it), scale by 1/l, store
            if (my_count > 0) {
                if (!warp_wait(&o_done[t], (co + my_commits - 1) & 1, abort_flag, p.status, 13)) break;
                tc_fence_after();
                const float inv = 1.f / l_sum;
                uint8_t* orow = reinterpret_cast<uint8_t*>(p.O + (static_cast<size_t>(g.bh) * p.S + row_g) * kD);
                // two rounds of 64 columns: both TMEM loads of a round in flight, then 32-byte stores (a lane
                // fills whole sectors; a 16-byte store pattern leaves every sector half written per instruction)
#pragma unroll 1
                for (int half = 0; half < 2; ++half) {
                    uint32_t ov[2][32];
                    tmem_ld32(tO + half * 64, ov[0]);
                    tmem_ld32(tO + half * 64 + 32, ov[1]);
                    tmem_wait_ld();
                    if (row_g < p.S) {
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            uint32_t pk[16];
#pragma unroll
                            for (int i = 0; i < 16; ++i)
                                pk[i] = pack_bf16x2(__uint_as_float(ov[c][2 * i]) * inv, __uint_as_float(ov[c][2 * i + 1]) * inv);
                            uint8_t* dst = orow + half * 128 + c * 64;
                            if (p.o_vec8) {
                                st_global_v8(dst, &pk[0]);
                                st_global_v8(dst + 32, &pk[8]);
                            } else {
#pragma unroll
                                for (int v = 0; v < 4; ++v)
                                    reinterpret_cast<uint4*>(dst)[v] = make_uint4(pk[4 * v], pk[4 * v + 1], pk[4 * v + 2], pk[4 * v + 3]);
                            }
                        }
                    }
                }
                co += static_cast<uint32_t>(my_commits);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&o_free[t]);   // every item, also when this tile had no work
            ++n_items;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace attn
}  // namespace ef

extern "C" {

size_t ef_qknorm_attn_workspace_bytes(int B, int H, int S, int D) {
    if (B <= 0 || H <= 0 || S <= 0 || D != ef::attn::kD) return 0;
    return ef::kDataOffset + static_cast<size_t>(B) * H * S * D * 2;   // header window + Khat (normalised keys, fp16)
}

ef_status ef_qknorm_attn_ex(const void* Q, const void* K, const void* V, const void* gamma_q, const void* gamma_k, void* O,
                            int B, int Hq, int Hkv, int S, int D, float eps, float scale, int causal, int window, int sinks,
                            void* ws, size_t ws_bytes, void* stream) {
    using namespace ef;
    if (!Q || !K || !V || !gamma_q || !gamma_k || !O) return EF_ERR_NULL;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || S <= 0 || D <= 0 || Hq % Hkv != 0 || window < 0 || sinks < 0) return EF_ERR_SHAPE;
    if (D != attn::kD || !(scale > 0.f)) return EF_ERR_UNSUPPORTED;
    if ((window > 0 || sinks > 0) && !causal) return EF_ERR_UNSUPPORTED;   // the window is defined for causal attention
    if (sinks > attn::kT || (sinks > 0 && window == 0)) return EF_ERR_UNSUPPORTED;   // sink keys lie in the first key tile
    const long long BH = static_cast<long long>(B) * Hq;
    const long long BHkv = static_cast<long long>(B) * Hkv;
    const int nq = (S + attn::kT - 1) / attn::kT;
    const int n_pairs = (nq + 1) / 2;
    if (BH * n_pairs > 0x7fffffffLL || BH > 0x3fffffff) return EF_ERR_UNSUPPORTED;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(gamma_q, 2) ||
        !aligned(gamma_k, 2))
        return EF_ERR_ALIGN;
    if (!ws || ws_bytes < ef_qknorm_attn_workspace_bytes(B, Hkv, S, D)) return EF_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return EF_ERR_ALIGN;
    DeviceInfo di;
    if (!current_device_info(&di)) return EF_ERR_CUDA;
    if (di.cc_major != 10) return EF_ERR_ARCH;

    CUtensorMap tmQ, tmK, tmV;
    const uint64_t dims[3] = {static_cast<uint64_t>(D), static_cast<uint64_t>(S), static_cast<uint64_t>(BH)};
    const uint64_t kdims[3] = {static_cast<uint64_t>(D), static_cast<uint64_t>(S), static_cast<uint64_t>(BHkv)};
    const uint64_t strides[2] = {static_cast<uint64_t>(D) * 2, static_cast<uint64_t>(S) * D * 2};
    const uint32_t box[3] = {64, attn::kT, 1};
    ef_status st;
    if ((st = encode_tmap_bf16(&tmQ, Q, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    uint8_t* w = static_cast<uint8_t*>(ws);
    __nv_bfloat16* Khat = reinterpret_cast<__nv_bfloat16*>(w + kDataOffset);
    if ((st = encode_tmap_bf16(&tmK, Khat, 3, kdims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    if ((st = encode_tmap_bf16(&tmV, V, 3, kdims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;

    static bool attr_set[64] = {};
    if (!attr_set[di.device]) {
        EF_CUDA_CHECK(cudaFuncSetAttribute(attn::qknorm_attn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           attn::kSmemBytes));
        EF_CUDA_CHECK(cudaFuncSetAttribute(attn::qknorm_attn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           attn::kSmemBytes));
        attr_set[di.device] = true;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    {
        const long long rows = BHkv * S;
        const long long blocks = (rows + 16 * attn::kKeyRowsPerThread - 1) / (16 * attn::kKeyRowsPerThread);
        if (blocks > 0x7fffffffLL) return EF_ERR_UNSUPPORTED;
        EF_CUDA_CHECK(launch_pdl(attn::key_normalize_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, s,
                                 static_cast<const __nv_bfloat16*>(K), static_cast<const __nv_bfloat16*>(gamma_q),
                                 static_cast<const __nv_bfloat16*>(gamma_k), Khat, rows, eps));
    }
    attn::Params p;
    p.gamma_q = static_cast<const __nv_bfloat16*>(gamma_q);
    p.gamma_k = static_cast<const __nv_bfloat16*>(gamma_k);
    p.O = static_cast<__nv_bfloat16*>(O);
    p.BH = static_cast<int>(BH); p.S = S; p.nq = nq; p.n_pairs = n_pairs; p.causal = causal ? 1 : 0;
    p.Hq = Hq; p.Hkv = Hkv;
    p.window = (window >= S) ? 0 : window;   // a window that covers every key is no window
    p.sinks = p.window > 0 ? sinks : 0;
    p.eps = eps;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = reinterpret_cast<uint32_t*>(w);
    p.header = reinterpret_cast<uint32_t*>(w);
    p.total_items = static_cast<int>(BH * n_pairs);
    p.o_vec8 = aligned(O, 32) ? 1 : 0;
    const unsigned grid = static_cast<unsigned>(p.total_items < di.num_sms ? p.total_items : di.num_sms);
    if (p.window > 0)
        EF_CUDA_CHECK(launch_pdl(attn::qknorm_attn_kernel<true>, dim3(grid), dim3(attn::kThreads), attn::kSmemBytes, s, tmQ, tmK, tmV, p));
    else
        EF_CUDA_CHECK(launch_pdl(attn::qknorm_attn_kernel<false>, dim3(grid), dim3(attn::kThreads), attn::kSmemBytes, s, tmQ, tmK, tmV, p));
    return EF_OK;
}

ef_status ef_qknorm_attn(const void* Q, const void* K, const void* V, const void* gamma_q, const void* gamma_k, void* O,
                         int B, int H, int S, int D, float eps, float scale, int causal, void* ws, size_t ws_bytes,
                         void* stream) {
    return ef_qknorm_attn_ex(Q, K, V, gamma_q, gamma_k, O, B, H, H, S, D, eps, scale, causal, 0, 0, ws, ws_bytes, stream);
}

}  // extern "C"
