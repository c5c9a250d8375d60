// ef_gqa_decode: grouped-query decode attention (one query token, L cached keys), HBM-bound.
//
// Execution form (Figure 4, M2 + Section 4.4): the key axis is tiled into chunks of 128 keys.
// The chunks of all (batch, kv-head) units form one list that is split into contiguous ranges,
// one per persistent thread block (grid = #SMs).  Inside a block the chunks of a range are
// traversed by a loop that carries the rolling state <max, sum, value> (the parallel reduce axis
// becomes an in-block loop, Section 6.1); where a unit's chunks are spread over several blocks the
// partial states are stored (Collection) and merged by the block that arrives last, using the same
// associative reducer, in block order (deterministic, no floating-point atomics).
//
// Data movement: a producer thread streams K and V chunks with TMA (128-byte swizzle) through a
// 3-stage, 64 KiB-per-stage shared-memory ring, so ~192 KiB per SM are in flight (a plain
// streaming kernel with this ring reads 128 MiB in ~25 us on a B200; stages of 16 KiB or less lose
// 15-40 % of that).  Four consumer warps each own 32 keys of every chunk: QK^T and PV run on
// warp-level mma.sync (the <= 8 query heads that share a kv head are the M rows of the MMA),
// softmax statistics are reduced with warp shuffles.  The kernel moves 2 bytes per 4 flops;
// tcgen05 would not help it.  All index arithmetic on the merge path is 32-bit: a 64-bit division
// per element there once cost more than the whole data stream.
#include <mutex>

#include "host.cuh"
#include "ptx.cuh"

namespace ef {
namespace decode {

constexpr int kD = 128;
constexpr int kChunk = 128;                       // keys per pipeline stage
constexpr int kStages = 3;
constexpr int kHalfBytes = kChunk * 128;          // [128 keys][64 dims] bf16, 128B-swizzled
constexpr int kStageBytes = 4 * kHalfBytes;       // K lo, K hi, V lo, V hi
constexpr int kConsumerWarps = 4;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;
constexpr int kKeysPerWarp = kChunk / kConsumerWarps;  // 32
constexpr int kMaxGroup = 8;                      // query heads per kv head (rows 0..7 of the MMA)
constexpr int kRowFloats = kD + 4;                // value[128], m, l, 2 pad (rows stay 16-byte aligned)
constexpr int kSlotFloats = kMaxGroup * kRowFloats;
constexpr int kMergeBytes = kConsumerWarps * kSlotFloats * 4;
constexpr int kMaxGrid = 256;                     // upper bound on the persistent grid
constexpr int kBarBytes = 128 + kMaxGrid * 4;     // barriers, flags, slot table of the final merge
constexpr int kMaxVarlenB = 1024;                 // batch entries of the per-sequence-length variant
constexpr int kCumBytes = (2 * kMaxVarlenB + 4) * 4;   // chunk-count prefix over the batch, base/rem, clamped lengths (that variant only)
constexpr int kSmemBytes = 1024 /*align slack*/ + kStages * kStageBytes + kMergeBytes + kBarBytes + kCumBytes;

struct Params {
    const __nv_bfloat16* Q;
    __nv_bfloat16* O;
    int B, Hq, Hkv, L, G;
    // sliding window + attention sinks (uniform-length kernel only; all zero = no window): the list of a unit is
    // sink_chunks leading chunks followed by the chunks from win_chunk0 on; key j counts iff j >= win_start or j < sinks
    int win_start, sinks, sink_chunks, win_chunk0;
    const int* seq_lens;   // per-sequence-length variant: keys [0, seq_lens[b]) of batch entry b are attended
    int n_chunks;      // chunks per (b, kv head) unit (uniform variant)
    int total_items;   // units * n_chunks  (< 2^30)
    int base, rem;     // block c owns base + (c < rem) consecutive items
    float scale_log2;  // scale * log2(e)
    uint32_t* status;
    uint32_t* counters;  // one arrival counter per unit, zero between calls
    float* partials;     // [grid][2][kMaxGroup][kRowFloats]
};

// Warp-uniform bounded wait: every lane polls, the warp proceeds only if all lanes succeeded.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status, uint32_t site) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, status, site)) != 0;
}
__device__ __forceinline__ void consumer_sync() {
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
}
// Contiguous partition of the item list (32-bit arithmetic only).
__device__ __forceinline__ int range_begin(int c, int base, int rem) { return c * base + min(c, rem); }
__device__ __forceinline__ int owner_of(int x, int base, int rem) {
    const int big = rem * (base + 1);
    return x < big ? x / (base + 1) : rem + (x - big) / base;
}
// Where item x of the flattened chunk list lies.  Uniform lengths: every (batch, kv head) unit has n_chunks chunks.
// Per-sequence lengths: a unit of batch entry b has nb_b = ceil(len_b / 128) chunks FOLLOWED BY ONE EMPTY ITEM (the
// fixed per-unit cost -- query load, four-warp merge, output write -- is about one chunk's worth of time, and equal
// item counts per block should mean equal time: a block that gets many one-chunk sequences gets half as many);
// cum[b] = sum of (nb + 1) over earlier entries with keys, and the Hkv units of an entry follow each other, so entry b
// owns items [Hkv*cum[b], Hkv*cum[b+1]).
// Layout of `cum` (shared memory, per-sequence-length variant only): [0..B] prefix, [B+1] base, [B+2] rem,
// [B+3 ..] clamped lengths.
struct Where {
    int unit;         // b * Hkv + kv head
    int chunk;        // chunk of x within the unit
    int unit_begin;   // item index of the unit's first chunk
    int n_chunks;     // chunks of the unit
    int n_items;      // items of the unit in the list (n_chunks, plus the empty item of the per-sequence-length variant)
    int len;          // keys of the unit
};
template <bool VARLEN>
__device__ __forceinline__ Where locate(int x, const Params& p, const int* cum) {
    Where w;
    if (!VARLEN) {
        w.unit = x / p.n_chunks;
        w.unit_begin = w.unit * p.n_chunks;
        w.chunk = x - w.unit_begin;
        w.n_chunks = p.n_chunks;
        w.n_items = p.n_chunks;
        w.len = p.L;
    } else {
        int lo = 0, hi = p.B;   // largest b with Hkv * cum[b] <= x (entries without keys own no items)
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (p.Hkv * cum[mid] <= x) lo = mid; else hi = mid;
        }
        const int nb = cum[lo + 1] - cum[lo];
        const int rel = x - p.Hkv * cum[lo];
        const int kvh = rel / nb;
        w.unit = lo * p.Hkv + kvh;
        w.chunk = rel - kvh * nb;
        w.unit_begin = x - w.chunk;
        w.n_chunks = nb - 1;
        w.n_items = nb;
        w.len = cum[p.B + 3 + lo];   // clamped length, cached by the prologue
    }
    return w;
}
// Partial-state slot of block c for `unit`: 0 if the unit is the first one the block touches, else 1.
template <bool VARLEN>
__device__ __forceinline__ int slot_of(int c, int unit, int base, int rem, const Params& p, const int* cum) {
    return 2 * c + (locate<VARLEN>(range_begin(c, base, rem), p, cum).unit == unit ? 0 : 1);
}

template <bool VARLEN, bool WIN>
__global__ void __launch_bounds__(kThreads, 1)
gqa_decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* stages = smem;
    float* merge = reinterpret_cast<float*>(smem + kStages * kStageBytes);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes + kMergeBytes);
    uint64_t* fullK = bars;                 // [kStages]
    uint64_t* fullV = bars + kStages;       // [kStages]
    uint64_t* empty = bars + 2 * kStages;   // [kStages]
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 3 * kStages);
    uint32_t* is_last = const_cast<uint32_t*>(abort_flag) + 1;
    int* slot_table = reinterpret_cast<int*>(bars) + 32;  // [kMaxGrid]
    int* cum = reinterpret_cast<int*>(smem + kStages * kStageBytes + kMergeBytes + kBarBytes);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&fullK[s], 1);
            mbar_init(&fullV[s], 1);
            mbar_init(&empty[s], kConsumerWarps);
        }
        *abort_flag = 0u;
        *is_last = 0u;
        fence_mbar_init();
    }
    pdl_launch_dependents();
    __syncthreads();
    pdl_wait();  // everything below may touch global memory of the previous kernel in the stream

    int base = p.base, rem = p.rem;
    if (VARLEN) {
        // Every block builds the same chunk-count prefix over the batch (warp 0: a serial piece per lane, then a
        // shuffle scan of the lane totals) and derives the partition of the item list from its total.
        if (warp == 0) {
            const int per = (p.B + 31) / 32;
            const int b0 = lane * per;
            int sum = 0, longest = 0;   // items of this lane's entries; most items of one entry
            for (int i = 0; i < per; ++i) {
                const int b = b0 + i;
                if (b < p.B) {
                    int len = p.seq_lens[b];
                    len = len < 0 ? 0 : (len > p.L ? p.L : len);
                    cum[p.B + 3 + b] = len;
                    const int items = len > 0 ? (len + kChunk - 1) / kChunk + 1 : 0;
                    sum += items;
                    longest = longest > items ? longest : items;
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const int v = __shfl_xor_sync(0xffffffffu, longest, o);
                longest = longest > v ? longest : v;
            }
            int incl = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            int run = incl - sum;   // chunks of the entries before this lane's piece
            for (int i = 0; i < per; ++i) {
                const int b = b0 + i;
                if (b < p.B) {
                    cum[b] = run;
                    run += cum[p.B + 3 + b] > 0 ? (cum[p.B + 3 + b] + kChunk - 1) / kChunk + 1 : 0;
                }
            }
            if (lane == 31) {
                cum[p.B] = incl;
                const int total = incl * p.Hkv;
                cum[p.B + 1] = total / static_cast<int>(gridDim.x);
                cum[p.B + 2] = total % static_cast<int>(gridDim.x);
                // One block per whole (batch, kv head) unit needs no partial states and no merging block; it wins unless one
                // sequence is much longer than the average block's share (cost model from measurements: a block alone
                // streams a chunk in ~0.75 us, all blocks together one in ~0.0115 us, the partial exchange costs ~9 us
                // with a length mix): every block takes this decision from the same numbers.
                cum[2 * p.B + 3] = (p.B * p.Hkv <= static_cast<int>(gridDim.x) && longest < total / 65 + 12) ? 1 : 0;
            }
        }
        __syncthreads();
        base = cum[p.B + 1];
        rem = cum[p.B + 2];
        // entries without keys: softmax over nothing, the output row is defined as zero (block 0 writes it)
        if (blockIdx.x == 0) {
            for (int b = 0; b < p.B; ++b) {
                if (cum[b + 1] == cum[b]) {
                    for (int i = tid; i < p.Hq * (kD / 8); i += kThreads)
                        reinterpret_cast<uint4*>(p.O + static_cast<size_t>(b) * p.Hq * kD)[i] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
        }
    }
    int it_begin = range_begin(blockIdx.x, base, rem);
    int it_end = range_begin(blockIdx.x + 1, base, rem);
    if (VARLEN && cum[2 * p.B + 3]) {   // block = unit: every unit is whole, so the merge path below is never entered
        const int bb = static_cast<int>(blockIdx.x) / p.Hkv, kvh = static_cast<int>(blockIdx.x) - bb * p.Hkv;
        it_begin = it_end = 0;
        if (bb < p.B) {
            const int nb = cum[bb + 1] - cum[bb];
            it_begin = p.Hkv * cum[bb] + kvh * nb;
            it_end = it_begin + nb;
        }
    }

    if (warp == kConsumerWarps) {
        // ------------------------------ producer warp ------------------------------
        if (lane == 0) {
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmV);
            int stage = 0;
            uint32_t phase = 0;
            Where w = {0, 0, 0, 1, 1, 0};
            if (it_begin < it_end) w = locate<VARLEN>(it_begin, p, cum);
            int unit = w.unit, chunk = w.chunk, unit_chunks = w.n_chunks, unit_items = w.n_items;
            for (int it = it_begin; it < it_end; ++it) {
                if (chunk >= unit_chunks) {   // the unit's empty item: nothing to load
                    chunk = 0;
                    ++unit;
                    if (it + 1 < it_end) {
                        const Where nx = locate<VARLEN>(it + 1, p, cum);
                        unit = nx.unit;
                        unit_chunks = nx.n_chunks;
                        unit_items = nx.n_items;
                    }
                    continue;
                }
                if (!mbar_wait(&empty[stage], phase ^ 1u, abort_flag, p.status, 1)) break;
                uint8_t* st = stages + stage * kStageBytes;
                const int key0 = (WIN ? (chunk < p.sink_chunks ? chunk : p.win_chunk0 + chunk - p.sink_chunks) : chunk) * kChunk;
                mbar_expect_tx(&fullK[stage], 2 * kHalfBytes);
                tma_load_3d(st, &tmK, &fullK[stage], 0, key0, unit);
                tma_load_3d(st + kHalfBytes, &tmK, &fullK[stage], 64, key0, unit);
                mbar_expect_tx(&fullV[stage], 2 * kHalfBytes);
                tma_load_3d(st + 2 * kHalfBytes, &tmV, &fullV[stage], 0, key0, unit);
                tma_load_3d(st + 3 * kHalfBytes, &tmV, &fullV[stage], 64, key0, unit);
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
                if (++chunk == unit_items) {   // (uniform lengths: items == chunks; otherwise the empty item comes next)
                    chunk = 0;
                    ++unit;
                }
            }
        }
    } else {
        // ------------------------------ consumer warps -----------------------------
        const int g = lane >> 2;        // fragment row = query head within the group (rows 8..15 are padding)
        const int t4 = lane & 3;
        int stage = 0;
        uint32_t phase = 0;
        int it = it_begin;
        bool ok = true;
        while (it < it_end && ok) {
            const Where w = locate<VARLEN>(it, p, cum);
            const int unit = w.unit;
            const int c0 = w.chunk;
            const int unit_end = w.unit_begin + w.n_chunks;            // end of the unit's chunks in the list
            const int items_end = w.unit_begin + w.n_items;            // ... and of its items
            const int len = w.len;   // keys of this unit
            const int seg_stop = items_end < it_end ? items_end : it_end;   // where this block leaves the unit
            const int seg_end = unit_end < seg_stop ? unit_end : seg_stop;  // ... and its last chunk of the unit
            const int n_seg = seg_end - it;
            if (n_seg <= 0) {   // only the unit's empty item falls into this block's range
                it = seg_stop;
                continue;
            }
            const bool whole_unit = (c0 == 0) && (seg_end == unit_end);
            const int b = unit / p.Hkv, kvh = unit - b * p.Hkv;
            const int head0 = kvh * p.G;

            // Q fragments (A operand, 16 x 128): rows >= G are zero padding.
            uint32_t qf[8][4];
            {
                const uint32_t* q0 = reinterpret_cast<const uint32_t*>(p.Q + (static_cast<size_t>(b) * p.Hq + head0 + g) * kD);
                const bool r0 = g < p.G;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const int c = ks * 8 + t4;  // uint32 index of column ks*16 + 2*t4
                    qf[ks][0] = r0 ? __ldg(q0 + c) : 0u;
                    qf[ks][1] = 0u;
                    qf[ks][2] = r0 ? __ldg(q0 + c + 4) : 0u;
                    qf[ks][3] = 0u;
                }
            }
            float m_run = -INFINITY, l_run = 0.f;
            float o[16][4];
#pragma unroll
            for (int i = 0; i < 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }

            for (int ch = 0; ch < n_seg; ++ch) {
                const int kc = WIN ? ((c0 + ch) < p.sink_chunks ? (c0 + ch) : p.win_chunk0 + (c0 + ch) - p.sink_chunks) : (c0 + ch);   // key chunk of this item
                const int key_base = kc * kChunk + warp * kKeysPerWarp;
                const uint32_t st = smem_u32(stages + stage * kStageBytes);
                if (!warp_wait(&fullK[stage], phase, abort_flag, p.status, 2)) { ok = false; break; }
                // ---- S = Q K^T for this warp's 32 keys: 4 n-tiles x 8 k-steps
                float s[4][4];
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
                    s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
                    const int key_local = warp * kKeysPerWarp + nt * 8 + (lane & 7);
#pragma unroll
                    for (int kp = 0; kp < 4; ++kp) {
                        const int c = kp * 4 + (lane >> 3);  // 16-byte chunk along d, 0..15
                        const uint32_t addr = st + (c >> 3) * kHalfBytes + key_local * 128 +
                                              (((c & 7) ^ (key_local & 7)) << 4);
                        uint32_t kb[4];
                        ldmatrix_x4(kb, addr);
                        mma_bf16_16816(s[nt], qf[2 * kp], kb[0], kb[1]);
                        mma_bf16_16816(s[nt], qf[2 * kp + 1], kb[2], kb[3]);
                    }
                }
                // ---- rolling softmax state update (log2 domain), rows 0..7 only
                float mx = -INFINITY;
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
                    const int key = key_base + nt * 8 + 2 * t4;
                    const bool v0 = key < len && (!WIN || key >= p.win_start || key < p.sinks);
                    const bool v1 = key + 1 < len && (!WIN || key + 1 >= p.win_start || key + 1 < p.sinks);
                    s[nt][0] = v0 ? s[nt][0] * p.scale_log2 : -INFINITY;
                    s[nt][1] = v1 ? s[nt][1] * p.scale_log2 : -INFINITY;
                    mx = fmaxf(mx, fmaxf(s[nt][0], s[nt][1]));
                }
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run, mx);
                const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;  // identity state: avoid inf - inf
                const float resc = fast_exp2(m_run - m_safe);
                m_run = m_new;
                float sum = 0.f;
                uint32_t pf[2][4];
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
                    const float p0 = fast_exp2(s[nt][0] - m_safe), p1 = fast_exp2(s[nt][1] - m_safe);
                    sum += p0 + p1;
                    pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16x2(p0, p1);
                    pf[nt >> 1][(nt & 1) * 2 + 1] = 0u;
                }
                l_run = l_run * resc + sum;
#pragma unroll
                for (int i = 0; i < 16; ++i) { o[i][0] *= resc; o[i][1] *= resc; }
                // ---- value += P V for this warp's 32 keys: 2 k-steps x 16 n-tiles
                if (!warp_wait(&fullV[stage], phase, abort_flag, p.status, 3)) { ok = false; break; }
                if (VARLEN && (c0 + ch + 1) * kChunk > len) {
                    // Keys at and beyond the sequence length are padding that may hold anything (their weight
                    // is 0, but 0 * NaN is NaN): this warp zeroes its own padded V rows before reading them.
                    const int key_l = warp * kKeysPerWarp + lane;   // one row per lane
                    if ((c0 + ch) * kChunk + key_l >= len) {
                        uint8_t* vrow = stages + stage * kStageBytes + 2 * kHalfBytes + key_l * 128;
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            *reinterpret_cast<uint4*>(vrow + c * 16) = make_uint4(0u, 0u, 0u, 0u);
                            *reinterpret_cast<uint4*>(vrow + kHalfBytes + c * 16) = make_uint4(0u, 0u, 0u, 0u);
                        }
                    }
                    fence_proxy_async_smem();   // the stage is refilled by the async proxy later
                    __syncwarp();
                }
#pragma unroll
                for (int kk = 0; kk < 2; ++kk) {
                    const int key_local = warp * kKeysPerWarp + kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
                    for (int np = 0; np < 8; ++np) {
                        const int c = 2 * np + (lane >> 4);
                        const uint32_t addr = st + (2 + (c >> 3)) * kHalfBytes + key_local * 128 +
                                              (((c & 7) ^ (key_local & 7)) << 4);
                        uint32_t vb[4];
                        ldmatrix_x4_trans(vb, addr);
                        mma_bf16_16816(o[2 * np], pf[kk], vb[0], vb[1]);
                        mma_bf16_16816(o[2 * np + 1], pf[kk], vb[2], vb[3]);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[stage]);
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;

            // ---- merge the four warps' states for this segment
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
            if (g < p.G) {
                float* row = merge + warp * kSlotFloats + g * kRowFloats;
                if (t4 == 0) { row[kD] = m_run; row[kD + 1] = l_run; }
#pragma unroll
                for (int i = 0; i < 16; ++i) *reinterpret_cast<float2*>(row + i * 8 + 2 * t4) = make_float2(o[i][0], o[i][1]);
            }
            consumer_sync();
            float* pslot = p.partials + static_cast<size_t>(slot_of<VARLEN>(blockIdx.x, unit, base, rem, p, cum)) * kSlotFloats;
            for (int idx = tid; idx < p.G * kD; idx += kConsumerThreads) {
                const int r = idx >> 7, d = idx & (kD - 1);
                float mw[kConsumerWarps];
                float M = -INFINITY;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    mw[w] = merge[w * kSlotFloats + r * kRowFloats + kD];
                    M = fmaxf(M, mw[w]);
                }
                float acc = 0.f, lsum = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    const float sc = fast_exp2(mw[w] - M);  // a warp that saw no valid key has m = -inf -> 0
                    acc += sc * merge[w * kSlotFloats + r * kRowFloats + d];
                    lsum += sc * merge[w * kSlotFloats + r * kRowFloats + kD + 1];
                }
                if (whole_unit) {
                    p.O[(static_cast<size_t>(b) * p.Hq + head0 + r) * kD + d] = __float2bfloat16_rn(acc / lsum);
                } else {
                    pslot[r * kRowFloats + d] = acc;
                    if (d == 0) { pslot[r * kRowFloats + kD] = M; pslot[r * kRowFloats + kD + 1] = lsum; }
                }
            }
            if (!whole_unit) {
                // Collection + parallel reduce across blocks: the block that arrives last merges.
                __threadfence();
                consumer_sync();
                const int c_first = owner_of(w.unit_begin, base, rem);
                const int c_last = owner_of(unit_end - 1, base, rem);
                const int n_parts = c_last - c_first + 1;
                if (tid == 0) {
                    const uint32_t prev = atomicAdd(&p.counters[unit], 1u);
                    *is_last = (prev == static_cast<uint32_t>(n_parts - 1)) ? 1u : 0u;
                }
                for (int i = tid; i < n_parts; i += kConsumerThreads)
                    slot_table[i] = slot_of<VARLEN>(c_first + i, unit, base, rem, p, cum);
                consumer_sync();
                if (*is_last) {
                    __threadfence();
                    for (int idx = tid; idx < p.G * (kD / 4); idx += kConsumerThreads) {
                        const int r = idx >> 5, d4 = idx & 31;
                        float M = -INFINITY;
                        for (int i = 0; i < n_parts; ++i)
                            M = fmaxf(M, __ldcg(p.partials + static_cast<size_t>(slot_table[i]) * kSlotFloats + r * kRowFloats + kD));
                        float acc[4] = {0.f, 0.f, 0.f, 0.f};
                        float lsum = 0.f;
                        for (int i = 0; i < n_parts; ++i) {  // block order: deterministic
                            const float* ps = p.partials + static_cast<size_t>(slot_table[i]) * kSlotFloats + r * kRowFloats;
                            const float sc = fast_exp2(__ldcg(ps + kD) - M);
                            lsum += sc * __ldcg(ps + kD + 1);
                            const float4 v = __ldcg(reinterpret_cast<const float4*>(ps) + d4);
                            acc[0] += sc * v.x; acc[1] += sc * v.y; acc[2] += sc * v.z; acc[3] += sc * v.w;
                        }
                        const float inv = 1.f / lsum;
                        uint2 packed;
                        packed.x = pack_bf16x2(acc[0] * inv, acc[1] * inv);
                        packed.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
                        *reinterpret_cast<uint2*>(p.O + (static_cast<size_t>(b) * p.Hq + head0 + r) * kD + 4 * d4) = packed;
                    }
                    if (tid == 0) p.counters[unit] = 0u;  // leave the counter ready for the next call
                }
            }
            consumer_sync();  // merge buffer, slot table and is_last are reused by the next segment
            it = seg_stop;
        }
    }
    // Teardown.  On an aborted run give copies that are still in flight time to land before the
    // block (and its shared memory) goes away; the wait is bounded.
    __syncwarp();
    if (*abort_flag) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
}

}  // namespace decode
}  // namespace ef

extern "C" {

size_t ef_gqa_decode_workspace_bytes(int B, int Hq, int Hkv, int L, int D) {
    (void)Hq; (void)L; (void)D;
    if (B <= 0 || Hkv <= 0) return 0;
    return ef::kDataOffset + static_cast<size_t>(ef::decode::kMaxGrid) * 2 * ef::decode::kSlotFloats * sizeof(float);
}

ef_status ef_gqa_decode_window(const void* Q, const void* K, const void* V, void* O, int B, int Hq, int Hkv, int L, int D,
                               float scale, int window, int sinks, void* ws, size_t ws_bytes, void* stream) {
    using namespace ef;
    if (!Q || !K || !V || !O) return EF_ERR_NULL;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || L <= 0 || D <= 0 || Hq % Hkv != 0 || window < 0 || sinks < 0) return EF_ERR_SHAPE;
    if (D != decode::kD || Hq / Hkv > decode::kMaxGroup) return EF_ERR_UNSUPPORTED;
    const size_t n_units = static_cast<size_t>(B) * Hkv;
    const size_t counters_bytes = (n_units * sizeof(uint32_t) + 255) & ~size_t(255);
    if (kHeaderBytes + counters_bytes > 65536) return EF_ERR_UNSUPPORTED;  // counters must lie in the init window
    // The single query sits at position L - 1: with a window it sees keys j >= L - window and the first `sinks` keys.
    // Chunks between the sink chunks and the first window chunk are never loaded.
    const long long all_chunks = (static_cast<long long>(L) + decode::kChunk - 1) / decode::kChunk;
    int win_start = 0, sink_chunks = 0, win_chunk0 = 0;
    if (window > 0 && window < L) {
        win_start = L - window;
        win_chunk0 = win_start / decode::kChunk;
        sink_chunks = (sinks + decode::kChunk - 1) / decode::kChunk;
        if (sink_chunks > win_chunk0) sink_chunks = win_chunk0;
    }
    const long long n_chunks = sink_chunks + (all_chunks - win_chunk0);
    if (n_chunks * static_cast<long long>(n_units) >= (1LL << 30)) return EF_ERR_UNSUPPORTED;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16)) return EF_ERR_ALIGN;
    if (!ws || ws_bytes < ef_gqa_decode_workspace_bytes(B, Hq, Hkv, L, D)) return EF_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return EF_ERR_ALIGN;
    DeviceInfo di;
    if (!current_device_info(&di)) return EF_ERR_CUDA;
    if (di.cc_major != 10) return EF_ERR_ARCH;

    CUtensorMap tmK, tmV;
    const uint64_t dims[3] = {static_cast<uint64_t>(D), static_cast<uint64_t>(L), n_units};
    const uint64_t strides[2] = {static_cast<uint64_t>(D) * 2, static_cast<uint64_t>(L) * D * 2};
    const uint32_t box[3] = {64, decode::kChunk, 1};
    ef_status st = encode_tmap_bf16(&tmK, K, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != EF_OK) return st;
    st = encode_tmap_bf16(&tmV, V, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != EF_OK) return st;

    static bool attr_set[64] = {};
    if (!attr_set[di.device]) {
        EF_CUDA_CHECK(cudaFuncSetAttribute(decode::gqa_decode_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           decode::kSmemBytes));
        EF_CUDA_CHECK(cudaFuncSetAttribute(decode::gqa_decode_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           decode::kSmemBytes));
        attr_set[di.device] = true;
    }
    decode::Params p;
    p.Q = static_cast<const __nv_bfloat16*>(Q);
    p.O = static_cast<__nv_bfloat16*>(O);
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.L = L; p.G = Hq / Hkv;
    p.seq_lens = nullptr;
    p.win_start = win_start; p.sinks = win_start > 0 ? sinks : 0; p.sink_chunks = sink_chunks; p.win_chunk0 = win_chunk0;
    p.n_chunks = static_cast<int>(n_chunks);
    p.total_items = static_cast<int>(n_chunks * static_cast<long long>(n_units));
    int grid = di.num_sms < p.total_items ? di.num_sms : p.total_items;
    if (grid > decode::kMaxGrid) grid = decode::kMaxGrid;
    if (n_units <= static_cast<size_t>(grid) && win_start == 0) {
        // (With a window the visible keys of a unit are scattered over a long history and a block on its own streams
        // slower -- 34.5 us with 64 blocks against 30.0 us with 148 at B = 8, L = 32768, window 4096 -- so that case
        // keeps one block per SM.)
        // Fewer units than SMs: give every unit the same number s of blocks, chosen by a small cost model.  A unit that
        // is not split needs no partial state, no arrival counter and no merging block (measured: ~3.5 us at the end of
        // the kernel), and a block streams ~100 GB/s on its own, so 64 unsplit units already saturate HBM (B = 8:
        // 23.8 us with 64 blocks against 27.4 us with 148); few units (B = 1) must be split to use the machine.
        const double bytes = static_cast<double>(p.total_items) * decode::kStageBytes;
        const double hbm = 5.7e6, per_block = 0.1e6;   // bytes per microsecond
        double best = -1.0;
        int best_s = 1;
        for (int sp = 1; sp * static_cast<int>(n_units) <= grid && sp <= static_cast<int>(n_chunks); ++sp) {
            const double t_hbm = bytes / hbm, t_blk = bytes / (per_block * sp * static_cast<double>(n_units));
            // (a split that does not divide the chunk count makes ranges straddle units: more partial states per block;
            // measured at B = 1, 32 chunks: 8.7 us with 8 or 16 blocks per unit, 9.5 us with 18, 11.7 us with 12)
            const double t = (t_hbm > t_blk ? t_hbm : t_blk) + (sp > 1 ? 3.5 : 0.0) + (n_chunks % sp != 0 ? 1.5 : 0.0);
            if (best < 0.0 || t < best - 1e-9) { best = t; best_s = sp; }
        }
        grid = best_s * static_cast<int>(n_units);
    }
    p.base = p.total_items / grid;
    p.rem = p.total_items % grid;
    p.scale_log2 = scale * 1.4426950408889634f;
    uint8_t* w = static_cast<uint8_t*>(ws);
    p.status = reinterpret_cast<uint32_t*>(w);
    p.counters = reinterpret_cast<uint32_t*>(w + kHeaderBytes);
    p.partials = reinterpret_cast<float*>(w + kDataOffset);
    if (win_start > 0)
        EF_CUDA_CHECK(launch_pdl(decode::gqa_decode_kernel<false, true>, dim3(grid), dim3(decode::kThreads), decode::kSmemBytes,
                                 static_cast<cudaStream_t>(stream), tmK, tmV, p));
    else
        EF_CUDA_CHECK(launch_pdl(decode::gqa_decode_kernel<false, false>, dim3(grid), dim3(decode::kThreads), decode::kSmemBytes,
                                 static_cast<cudaStream_t>(stream), tmK, tmV, p));
    return EF_OK;
}

ef_status ef_gqa_decode(const void* Q, const void* K, const void* V, void* O, int B, int Hq, int Hkv, int L, int D,
                        float scale, void* ws, size_t ws_bytes, void* stream) {
    return ef_gqa_decode_window(Q, K, V, O, B, Hq, Hkv, L, D, scale, 0, 0, ws, ws_bytes, stream);
}

ef_status ef_gqa_decode_varlen(const void* Q, const void* K, const void* V, const void* seq_lens, void* O, int B, int Hq,
                               int Hkv, int Lmax, int D, float scale, void* ws, size_t ws_bytes, void* stream) {
    using namespace ef;
    if (!Q || !K || !V || !O || !seq_lens) return EF_ERR_NULL;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Lmax <= 0 || D <= 0 || Hq % Hkv != 0) return EF_ERR_SHAPE;
    if (D != decode::kD || Hq / Hkv > decode::kMaxGroup || B > decode::kMaxVarlenB) return EF_ERR_UNSUPPORTED;
    const size_t n_units = static_cast<size_t>(B) * Hkv;
    const size_t counters_bytes = (n_units * sizeof(uint32_t) + 255) & ~size_t(255);
    if (kHeaderBytes + counters_bytes > 65536) return EF_ERR_UNSUPPORTED;  // counters must lie in the init window
    const long long n_chunks = (static_cast<long long>(Lmax) + decode::kChunk - 1) / decode::kChunk;
    if (n_chunks * static_cast<long long>(n_units) >= (1LL << 30)) return EF_ERR_UNSUPPORTED;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(seq_lens, 4)) return EF_ERR_ALIGN;
    if (!ws || ws_bytes < ef_gqa_decode_workspace_bytes(B, Hq, Hkv, Lmax, D)) return EF_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return EF_ERR_ALIGN;
    DeviceInfo di;
    if (!current_device_info(&di)) return EF_ERR_CUDA;
    if (di.cc_major != 10) return EF_ERR_ARCH;

    CUtensorMap tmK, tmV;
    const uint64_t dims[3] = {static_cast<uint64_t>(D), static_cast<uint64_t>(Lmax), n_units};
    const uint64_t strides[2] = {static_cast<uint64_t>(D) * 2, static_cast<uint64_t>(Lmax) * D * 2};
    const uint32_t box[3] = {64, decode::kChunk, 1};
    ef_status st = encode_tmap_bf16(&tmK, K, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != EF_OK) return st;
    st = encode_tmap_bf16(&tmV, V, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != EF_OK) return st;

    static bool attr_set[64] = {};
    if (!attr_set[di.device]) {
        EF_CUDA_CHECK(cudaFuncSetAttribute(decode::gqa_decode_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           decode::kSmemBytes));
        attr_set[di.device] = true;
    }
    decode::Params p;
    p.Q = static_cast<const __nv_bfloat16*>(Q);
    p.O = static_cast<__nv_bfloat16*>(O);
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.L = Lmax; p.G = Hq / Hkv;
    p.seq_lens = static_cast<const int*>(seq_lens);
    p.win_start = 0; p.sinks = 0; p.sink_chunks = 0; p.win_chunk0 = 0;
    p.n_chunks = static_cast<int>(n_chunks);
    p.total_items = 0;   // the lengths live on the device: every block derives the item list and its range itself
    p.base = 0;
    p.rem = 0;
    const long long max_items = n_chunks * static_cast<long long>(n_units);
    int grid = di.num_sms < max_items ? di.num_sms : static_cast<int>(max_items);
    if (grid > decode::kMaxGrid) grid = decode::kMaxGrid;
    p.scale_log2 = scale * 1.4426950408889634f;
    uint8_t* w = static_cast<uint8_t*>(ws);
    p.status = reinterpret_cast<uint32_t*>(w);
    p.counters = reinterpret_cast<uint32_t*>(w + kHeaderBytes);
    p.partials = reinterpret_cast<float*>(w + kDataOffset);
    EF_CUDA_CHECK(launch_pdl(decode::gqa_decode_kernel<true, false>, dim3(grid), dim3(decode::kThreads), decode::kSmemBytes,
                             static_cast<cudaStream_t>(stream), tmK, tmV, p));
    return EF_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// ef_gqa_decode_static: the same decode attention for callers that cannot allocate
// ---------------------------------------------------------------------------------------------
// Scratch for this entry point lives in the library image: every GPU that loads the library
// holds these bytes until the process exits.  Layout = an ordinary decode workspace (header,
// one arrival counter per (batch, kv head) unit, partial-state slots of the persistent grid).
namespace ef {
namespace decode {
constexpr int kStaticMaxUnits = 1024;  // B * Hkv accepted by ef_gqa_decode_static
constexpr size_t kStaticScratchBytes = kDataOffset + static_cast<size_t>(kMaxGrid) * 2 * kSlotFloats * sizeof(float);
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
// On the host, `g_static_scratch` is only a handle for the runtime, not a device address; the
// address the kernel needs is looked up once per device and cached here.
static void* g_static_scratch_ptr[64] = {};
static std::mutex g_static_mu;
}  // namespace decode
}  // namespace ef

extern "C" {

size_t ef_gqa_decode_static_max_units(void) { return ef::decode::kStaticMaxUnits; }

ef_status ef_gqa_decode_static(const void* Q, const void* K, const void* V, void* O, int B, int Hq, int Hkv, int L, int D,
                               float scale, void* stream) {
    using namespace ef;
    if (B <= 0 || Hkv <= 0) return EF_ERR_SHAPE;
    if (static_cast<long long>(B) * Hkv > decode::kStaticMaxUnits) return EF_ERR_WORKSPACE;  // beyond the built-in scratch
    int dev = -1;
    EF_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return EF_ERR_UNSUPPORTED;
    void* ptr = nullptr;
    {
        std::lock_guard<std::mutex> lk(decode::g_static_mu);
        if (!decode::g_static_scratch_ptr[dev]) {
            // first call on this device (which is current): resolve the array's device address
            void* p = nullptr;
            EF_CUDA_CHECK(cudaGetSymbolAddress(&p, decode::g_static_scratch));
            decode::g_static_scratch_ptr[dev] = p;
        }
        ptr = decode::g_static_scratch_ptr[dev];
    }
    // The array keeps whatever the previous call left: status word and arrival counters must start at zero.
    EF_CUDA_CHECK(cudaMemsetAsync(ptr, 0, kHeaderBytes + decode::kStaticMaxUnits * sizeof(uint32_t),
                                  static_cast<cudaStream_t>(stream)));
    return ef_gqa_decode(Q, K, V, O, B, Hq, Hkv, L, D, scale, ptr, decode::kStaticScratchBytes, stream);
}

}  // extern "C"
