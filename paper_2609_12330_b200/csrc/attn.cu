// ef_qknorm_attn: (causal) prefill attention with RMS-normalised queries and keys.
//
// Algebra (Table 1, factor motion; Section 7.3, QK-normalized MLA): with rq_i, rk_j the inverse
// RMS of query row i / key row j,
//     s_ij = scale * rq_i * rk_j * sum_d q_id (gq_d gk_d) k_jd ,
// so raw K tiles go TMA -> tensor core untouched, the gamma product is folded into the Q tile
// once per block, rk_j multiplies the logits column-wise and rq_i * scale * log2(e) row-wise.
// rk (one float per key) is produced by a small pre-pass kernel; rq is computed in the block.
//
// Execution form (Figure 4, M2): grid over (batch*head, pair of 128-row Q tiles) = axis m, loop
// over 128-key K/V tiles = axis p, rolling state <max, sum, value> with the repair
// h(c,s,s') = c * exp(s - s').  The repair is applied lazily: the accumulated value is rescaled
// only when the running maximum grows by more than 2^8 (any reference maximum is exact in real
// arithmetic because numerator and normaliser use the same one).  Causal: tiles above the
// diagonal are never visited, only the diagonal tile is masked.
//
// Pipeline per block (320 threads): warp 0 = TMA producer (Q once, K/V/rk rings), warp 1 = single
// thread issuing tcgen05.mma (S_t = Q_t K^T into TMEM, O_t += P_t V with P read from TMEM), warps
// 2..5 / 6..9 = softmax groups for Q tile 0 / 1 (one thread per row: tcgen05.ld S, exp2, write
// P as bf16 back into the S columns, rescale O when needed, final O / l).  While one group runs
// its softmax the tensor core works on the other tile.  Score and probability matrices never
// leave the SM (Section 7.2).
#include "host.cuh"
#include "ptx.cuh"

namespace ef {
namespace attn {

constexpr int kD = 128;
constexpr int kT = 128;                           // tile edge (queries and keys)
constexpr int kHalfBytes = kT * 128;              // [128 rows][64 d] bf16, 128B swizzle
constexpr int kTileBytes = 2 * kHalfBytes;        // 32 KiB
constexpr int kKVStages = 2;
constexpr int kThreads = 320;
constexpr int kSoftmaxThreads = 128;
constexpr uint32_t kTmemCols = 512;               // S0 | S1 | O0 | O1, 128 fp32 columns each
constexpr int kRkBytes = kT * 4;
// shared memory map (offsets from the 1024-aligned base)
constexpr int kOffQ = 0;                                          // 2 tiles
constexpr int kOffK = kOffQ + 2 * kTileBytes;                     // kKVStages tiles
constexpr int kOffV = kOffK + kKVStages * kTileBytes;             // kKVStages tiles
constexpr int kOffRk = kOffV + kKVStages * kTileBytes;            // [2 groups][2 stages][128 floats]
constexpr int kOffGamma = kOffRk + 2 * 2 * kRkBytes;              // [128 floats] gq*gk
constexpr int kOffBars = kOffGamma + kD * 4;
constexpr int kSmemBytes = 1024 + kOffBars + 512;
constexpr float kRescaleThreshold = 8.0f;         // log2 units

struct Params {
    const __nv_bfloat16* gamma_q;
    const __nv_bfloat16* gamma_k;
    const float* rk;      // [BH][s_pad]
    __nv_bfloat16* O;     // [BH][S][128]
    int BH, S, s_pad, nq, n_pairs, causal;
    float eps, scale_log2;
    uint32_t* status;
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

// ---------------------------------------------------------------------------------------------
// pre-pass: rk[bh][j] = rsqrt(mean_d K[bh][j][d]^2 + eps); 16 threads per key row
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) key_rms_kernel(const __nv_bfloat16* __restrict__ K, float* __restrict__ rk, int BH,
                                                      int S, int s_pad, float eps) {
    const long long total = static_cast<long long>(BH) * s_pad;
    const int sub = threadIdx.x & 15;
    for (long long row = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 4; row < total;
         row += (static_cast<long long>(gridDim.x) * blockDim.x) >> 4) {
        const int bh = static_cast<int>(row / s_pad), j = static_cast<int>(row - static_cast<long long>(bh) * s_pad);
        float ss = 0.f;
        if (j < S) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(K + (static_cast<size_t>(bh) * S + j) * kD) + sub);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float a = __uint_as_float(w[i] << 16), b = __uint_as_float(w[i] & 0xFFFF0000u);
                ss += a * a + b * b;
            }
        }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (sub == 0) rk[row] = (j < S) ? rsqrtf(ss * (1.f / kD) + eps) : 0.f;
    }
}

// ---------------------------------------------------------------------------------------------
// main kernel
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1)
qknorm_attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    float* gprod = reinterpret_cast<float*>(smem + kOffGamma);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kOffBars);
    uint64_t* q_full = bars;                 // [1]
    uint64_t* q_ready = bars + 1;            // [2]  softmax group -> MMA (Q tile rewritten)
    uint64_t* k_full = bars + 3;             // [2]
    uint64_t* k_empty = bars + 5;            // [2]
    uint64_t* v_full = bars + 7;             // [2]
    uint64_t* v_empty = bars + 9;            // [2]
    uint64_t* s_full = bars + 11;            // [2]  MMA -> softmax group t
    uint64_t* p_full = bars + 13;            // [2]  softmax group t -> MMA
    uint64_t* o_done = bars + 15;            // [2]  MMA -> softmax group t (PV finished)
    uint64_t* rk_full = bars + 17;           // [2 groups][2 stages]
    uint64_t* rk_empty = bars + 21;          // [2 groups][2 stages]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 25);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // heaviest (latest) Q tile pairs first: blocks are dispatched in index order
    const int pair = p.n_pairs - 1 - static_cast<int>(blockIdx.x / p.BH);
    const int bh = static_cast<int>(blockIdx.x % p.BH);
    const int qt0 = 2 * pair, qt1 = 2 * pair + 1;
    const bool has_q1 = qt1 < p.nq;
    const int q_last = has_q1 ? qt1 : qt0;
    const int n_kv = p.causal ? (q_last + 1) : p.nq;
    // number of key tiles each Q tile visits
    const int n_kv_t0 = p.causal ? (qt0 + 1) : p.nq;
    const int n_kv_t1 = has_q1 ? (p.causal ? (qt1 + 1) : p.nq) : 0;

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int t = 0; t < 2; ++t) {
            mbar_init(&q_ready[t], kSoftmaxThreads);
            mbar_init(&k_full[t], 1); mbar_init(&k_empty[t], 1);
            mbar_init(&v_full[t], 1); mbar_init(&v_empty[t], 1);
            mbar_init(&s_full[t], 1); mbar_init(&p_full[t], 4); mbar_init(&o_done[t], 1);
        }
        for (int i = 0; i < 4; ++i) { mbar_init(&rk_full[i], 1); mbar_init(&rk_empty[i], 4); }
        *abort_flag = 0u;
        fence_mbar_init();
    }
    if (threadIdx.x >= 64 && threadIdx.x < 64 + kD) {
        const int d = threadIdx.x - 64;
        gprod[d] = __bfloat162float(p.gamma_q[d]) * __bfloat162float(p.gamma_k[d]);
    }
    if (warp == 1) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
            mbar_expect_tx(q_full, 2 * kTileBytes);
            for (int t = 0; t < 2; ++t) {   // rows beyond S are out of bounds -> zero fill
                tma_load_3d(smem + kOffQ + t * kTileBytes, &tmQ, q_full, 0, (qt0 + t) * kT, bh);
                tma_load_3d(smem + kOffQ + t * kTileBytes + kHalfBytes, &tmQ, q_full, 64, (qt0 + t) * kT, bh);
            }
            bool ok = true;
            for (int j = 0; j < n_kv && ok; ++j) {
                const int st = j & 1;
                const uint32_t ph = ((j >> 1) & 1) ^ 1u;
                if (!mbar_wait(&k_empty[st], ph, abort_flag, p.status, 1)) break;
                mbar_expect_tx(&k_full[st], kTileBytes);
                tma_load_3d(smem + kOffK + st * kTileBytes, &tmK, &k_full[st], 0, j * kT, bh);
                tma_load_3d(smem + kOffK + st * kTileBytes + kHalfBytes, &tmK, &k_full[st], 64, j * kT, bh);
                for (int t = 0; t < 2; ++t) {
                    if (j >= (t == 0 ? n_kv_t0 : n_kv_t1)) continue;
                    if (!mbar_wait(&rk_empty[t * 2 + st], ph, abort_flag, p.status, 2)) { ok = false; break; }
                    mbar_expect_tx(&rk_full[t * 2 + st], kRkBytes);
                    bulk_load_1d(smem + kOffRk + (t * 2 + st) * kRkBytes, p.rk + static_cast<size_t>(bh) * p.s_pad + j * kT,
                                 kRkBytes, &rk_full[t * 2 + st]);
                }
                if (!ok) break;
                if (!mbar_wait(&v_empty[st], ph, abort_flag, p.status, 3)) break;
                mbar_expect_tx(&v_full[st], kTileBytes);
                tma_load_3d(smem + kOffV + st * kTileBytes, &tmV, &v_full[st], 0, j * kT, bh);
                tma_load_3d(smem + kOffV + st * kTileBytes + kHalfBytes, &tmV, &v_full[st], 64, j * kT, bh);
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            constexpr uint32_t idesc_qk = make_idesc_bf16(kT, kT, 0, 0);  // A = Q (K-major), B = K (K-major)
            constexpr uint32_t idesc_pv = make_idesc_bf16(kT, kD, 0, 1);  // A = P (TMEM),    B = V (MN-major)
            const uint32_t sQ = smem_u32(smem + kOffQ), sK = smem_u32(smem + kOffK), sV = smem_u32(smem + kOffV);
            auto issue_qk = [&](int t, int st) {
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
                    umma_ss(tmem_base + t * kT, make_smem_desc(sQ + t * kTileBytes + off, 16, 1024, kSwizzle128B),
                            make_smem_desc(sK + st * kTileBytes + off, 16, 1024, kSwizzle128B), idesc_qk, kk != 0 ? 1u : 0u);
                }
            };
            auto issue_pv = [&](int t, int st, uint32_t accumulate) {
#pragma unroll
                for (int kk = 0; kk < kT / 16; ++kk) {
                    umma_ts(tmem_base + 2 * kT + t * kD, tmem_base + t * kT + kk * 8,
                            make_smem_desc(sV + st * kTileBytes + kk * 2048, kHalfBytes, 1024, kSwizzle128B), idesc_pv,
                            (accumulate | static_cast<uint32_t>(kk)) != 0 ? 1u : 0u);
                }
            };
            const int nkv[2] = {n_kv_t0, n_kv_t1};
            bool ok = true;
            for (int t = 0; t < 2 && ok; ++t)
                if (nkv[t] > 0) ok = mbar_wait(&q_ready[t], 0u, abort_flag, p.status, 4);
            // S_t(0)
            if (ok) ok = mbar_wait(&k_full[0], 0u, abort_flag, p.status, 5);
            if (ok) {
                tc_fence_after();
                for (int t = 0; t < 2; ++t)
                    if (nkv[t] > 0) { issue_qk(t, 0); umma_commit(&s_full[t]); }
                umma_commit(&k_empty[0]);
            }
            for (int j = 0; j < n_kv && ok; ++j) {
                const int st = j & 1, stn = (j + 1) & 1;
                bool v_waited = false, k_waited = false;
                for (int t = 0; t < 2 && ok; ++t) {
                    if (j >= nkv[t]) continue;
                    if (!mbar_wait(&p_full[t], j & 1, abort_flag, p.status, 6)) { ok = false; break; }
                    if (!v_waited) {
                        if (!mbar_wait(&v_full[st], (j >> 1) & 1, abort_flag, p.status, 7)) { ok = false; break; }
                        v_waited = true;
                    }
                    tc_fence_after();
                    issue_pv(t, st, j > 0 ? 1u : 0u);
                    umma_commit(&o_done[t]);
                    if (j + 1 < nkv[t]) {
                        if (!k_waited) {
                            if (!mbar_wait(&k_full[stn], ((j + 1) >> 1) & 1, abort_flag, p.status, 8)) { ok = false; break; }
                            k_waited = true;
                            tc_fence_after();
                        }
                        issue_qk(t, stn);
                        umma_commit(&s_full[t]);
                    }
                }
                if (!ok) break;
                umma_commit(&v_empty[st]);           // all PV of key tile j issued
                if (k_waited) umma_commit(&k_empty[stn]);  // all QK of key tile j+1 issued
            }
        }
    } else {
        // ------------------------------ softmax groups ------------------------------
        const int t = (warp - 2) >> 2;             // 0: Q tile 0, 1: Q tile 1
        const int q = warp & 3;                    // TMEM lane quadrant
        const int r = q * 32 + lane;               // row within the tile
        const int qt = qt0 + t;
        const int my_nkv = (t == 0) ? n_kv_t0 : n_kv_t1;
        const int row_g = qt * kT + r;             // query index within the sequence
        const uint32_t lane_sel = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t tS = tmem_base + t * kT + lane_sel;
        const uint32_t tO = tmem_base + 2 * kT + t * kD + lane_sel;
        bool ok = my_nkv > 0;
        float rq = 0.f;
        if (ok) ok = warp_wait(q_full, 0u, abort_flag, p.status, 9);
        if (ok) {
            // rq_i and the in-place rewrite q'_d = bf16(q_d * gq_d * gk_d)
            uint8_t* qrow = smem + kOffQ + t * kTileBytes + r * 128;
            float ss = 0.f;
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                uint4* ptr = reinterpret_cast<uint4*>(qrow + (c >> 3) * kHalfBytes + (((c & 7) ^ (r & 7)) << 4));
                const uint4 v = *ptr;
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                uint32_t o4[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float a = __uint_as_float(w[i] << 16), b = __uint_as_float(w[i] & 0xFFFF0000u);
                    ss += a * a + b * b;
                    o4[i] = pack_bf16x2(a * gprod[c * 8 + 2 * i], b * gprod[c * 8 + 2 * i + 1]);
                }
                *ptr = make_uint4(o4[0], o4[1], o4[2], o4[3]);
            }
            rq = rsqrtf(ss * (1.f / kD) + p.eps) * p.scale_log2;
            fence_proxy_async_smem();
            mbar_arrive(&q_ready[t]);
        }
        float m_ref = -INFINITY, l_sum = 0.f;
        for (int j = 0; j < my_nkv && ok; ++j) {
            const int st = j & 1;
            if (!warp_wait(&s_full[t], j & 1, abort_flag, p.status, 10)) { ok = false; break; }
            if (!warp_wait(&rk_full[t * 2 + st], (j >> 1) & 1, abort_flag, p.status, 11)) { ok = false; break; }
            tc_fence_after();
            uint32_t s[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, s[c]);
            tmem_wait_ld();
            const float4* rk4 = reinterpret_cast<const float4*>(smem + kOffRk + (t * 2 + st) * kRkBytes);
            const bool diag = p.causal && (j == qt);
            const int key0 = j * kT;
            float umax = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
#pragma unroll
                for (int i4 = 0; i4 < 8; ++i4) {
                    const float4 k4 = rk4[c * 8 + i4];
                    const float kk[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int col = c * 32 + i4 * 4 + e;
                        float u = __uint_as_float(s[c][i4 * 4 + e]) * kk[e];
                        const bool valid = (!diag || col <= r) && (key0 + col < p.S);
                        u = valid ? u : -INFINITY;
                        s[c][i4 * 4 + e] = __float_as_uint(u);
                        umax = fmaxf(umax, u);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&rk_empty[t * 2 + st]);
            // lazy repair of the running maximum
            const float m_tile = umax * rq;   // rq > 0
            float o_scale = 1.f;
            const bool need = m_tile > m_ref + kRescaleThreshold;
            if (need) {
                o_scale = fast_exp2(m_ref - m_tile);  // 0 on the first tile (m_ref = -inf)
                l_sum *= o_scale;
                m_ref = m_tile;
            }
            float tile_sum = 0.f;
            uint32_t pk[64];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float p0 = fast_exp2(fmaf(__uint_as_float(s[c][i]), rq, -m_ref));
                    const float p1 = fast_exp2(fmaf(__uint_as_float(s[c][i + 1]), rq, -m_ref));
                    tile_sum += p0 + p1;
                    pk[c * 16 + (i >> 1)] = pack_bf16x2(p0, p1);
                }
            }
            l_sum += tile_sum;
            // P (bf16) overwrites the first 64 columns of this thread's own S row
            {
                uint32_t (&lo)[32] = *reinterpret_cast<uint32_t (*)[32]>(&pk[0]);
                uint32_t (&hi)[32] = *reinterpret_cast<uint32_t (*)[32]>(&pk[32]);
                tmem_st32(tS, lo);
                tmem_st32(tS + 32, hi);
            }
            // rescale the accumulated value when some row of this warp moved its reference maximum
            if (j > 0 && __any_sync(0xffffffffu, need)) {
                if (!warp_wait(&o_done[t], (j - 1) & 1, abort_flag, p.status, 12)) { ok = false; break; }
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
        }
        if (ok && my_nkv > 0) {
            // epilogue: O / l
            if (warp_wait(&o_done[t], (my_nkv - 1) & 1, abort_flag, p.status, 13)) {
                tc_fence_after();
                const float inv = 1.f / l_sum;
                __nv_bfloat16* orow = p.O + (static_cast<size_t>(bh) * p.S + row_g) * kD;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t ov[32];
                    tmem_ld32(tO + c * 32, ov);
                    tmem_wait_ld();
                    if (row_g < p.S) {
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint4 o;
                            o.x = pack_bf16x2(__uint_as_float(ov[v * 8 + 0]) * inv, __uint_as_float(ov[v * 8 + 1]) * inv);
                            o.y = pack_bf16x2(__uint_as_float(ov[v * 8 + 2]) * inv, __uint_as_float(ov[v * 8 + 3]) * inv);
                            o.z = pack_bf16x2(__uint_as_float(ov[v * 8 + 4]) * inv, __uint_as_float(ov[v * 8 + 5]) * inv);
                            o.w = pack_bf16x2(__uint_as_float(ov[v * 8 + 6]) * inv, __uint_as_float(ov[v * 8 + 7]) * inv);
                            *reinterpret_cast<uint4*>(orow + c * 32 + v * 8) = o;
                        }
                    }
                }
            }
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
    (void)D;
    if (B <= 0 || H <= 0 || S <= 0) return 0;
    const size_t s_pad = (static_cast<size_t>(S) + ef::attn::kT - 1) / ef::attn::kT * ef::attn::kT;
    return ef::kHeaderBytes + static_cast<size_t>(B) * H * s_pad * sizeof(float);
}

ef_status ef_qknorm_attn(const void* Q, const void* K, const void* V, const void* gamma_q, const void* gamma_k, void* O,
                         int B, int H, int S, int D, float eps, float scale, int causal, void* ws, size_t ws_bytes,
                         void* stream) {
    using namespace ef;
    if (!Q || !K || !V || !gamma_q || !gamma_k || !O) return EF_ERR_NULL;
    if (B <= 0 || H <= 0 || S <= 0 || D <= 0) return EF_ERR_SHAPE;
    if (D != attn::kD) return EF_ERR_UNSUPPORTED;
    const long long BH = static_cast<long long>(B) * H;
    const int nq = (S + attn::kT - 1) / attn::kT;
    const int n_pairs = (nq + 1) / 2;
    if (BH * n_pairs > 0x7fffffffLL || BH > 0x3fffffff) return EF_ERR_UNSUPPORTED;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(gamma_q, 2) ||
        !aligned(gamma_k, 2))
        return EF_ERR_ALIGN;
    if (!ws || ws_bytes < ef_qknorm_attn_workspace_bytes(B, H, S, D)) return EF_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return EF_ERR_ALIGN;
    DeviceInfo di;
    if (!current_device_info(&di)) return EF_ERR_CUDA;
    if (di.cc_major != 10) return EF_ERR_ARCH;

    CUtensorMap tmQ, tmK, tmV;
    const uint64_t dims[3] = {static_cast<uint64_t>(D), static_cast<uint64_t>(S), static_cast<uint64_t>(BH)};
    const uint64_t strides[2] = {static_cast<uint64_t>(D) * 2, static_cast<uint64_t>(S) * D * 2};
    const uint32_t box[3] = {64, attn::kT, 1};
    ef_status st;
    if ((st = encode_tmap_bf16(&tmQ, Q, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    if ((st = encode_tmap_bf16(&tmK, K, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;
    if ((st = encode_tmap_bf16(&tmV, V, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) != EF_OK) return st;

    static bool attr_set[64] = {};
    if (!attr_set[di.device]) {
        EF_CUDA_CHECK(cudaFuncSetAttribute(attn::qknorm_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           attn::kSmemBytes));
        attr_set[di.device] = true;
    }
    uint8_t* w = static_cast<uint8_t*>(ws);
    float* rk = reinterpret_cast<float*>(w + kHeaderBytes);
    const int s_pad = nq * attn::kT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    {
        const long long rows = BH * s_pad;
        long long blocks = (rows * 16 + 255) / 256;
        const long long cap = static_cast<long long>(di.num_sms) * 16;
        if (blocks > cap) blocks = cap;
        attn::key_rms_kernel<<<static_cast<unsigned>(blocks), 256, 0, s>>>(static_cast<const __nv_bfloat16*>(K), rk,
                                                                          static_cast<int>(BH), S, s_pad, eps);
        EF_CUDA_CHECK(cudaGetLastError());
    }
    attn::Params p;
    p.gamma_q = static_cast<const __nv_bfloat16*>(gamma_q);
    p.gamma_k = static_cast<const __nv_bfloat16*>(gamma_k);
    p.rk = rk;
    p.O = static_cast<__nv_bfloat16*>(O);
    p.BH = static_cast<int>(BH); p.S = S; p.s_pad = s_pad; p.nq = nq; p.n_pairs = n_pairs; p.causal = causal ? 1 : 0;
    p.eps = eps;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = reinterpret_cast<uint32_t*>(w);
    const unsigned grid = static_cast<unsigned>(BH * n_pairs);
    attn::qknorm_attn_kernel<<<grid, attn::kThreads, attn::kSmemBytes, s>>>(tmQ, tmK, tmV, p);
    EF_CUDA_CHECK(cudaGetLastError());
    return EF_OK;
}

}  // extern "C"
