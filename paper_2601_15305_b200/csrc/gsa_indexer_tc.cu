// Gated lightning indexer (Eq. 7) on the 5th-generation tensor cores.
//
//   D[s, (t, j)] = k^I[s, :] . q^I[t, j, :]         tcgen05.mma, bf16 x bf16 -> fp32 in TMEM
//   I[t, s]      = sum_j w[t, j] * sigmoid(D[s, (t, j)] + b_j)      epilogue, in registers
//
// Orientation: keys are the M dimension (128 per tile = the 128 TMEM lanes), the N dimension is
// (query, indexer head) flattened, 256 columns = 256/H^I queries.  A thread of the epilogue owns
// one key: it reads that key's 256 accumulators, sums the H^I adjacent columns of each query
// after the sigmoid, and consecutive lanes write consecutive s of a score row (128-byte stores).
//
// A CTA works on one query group and a run of key tiles at or below the diagonal (tiles above
// it are never touched).  Warp roles: warp 0 feeds shared memory by TMA (k^I tiles through a
// ring of stages, the q^I tile once), warp 1 issues the MMAs and owns the TMEM allocation,
// warps 2..17 are the epilogue.  Two 256-column accumulators alternate, so the MMAs of tile i+1
// overlap the epilogue of tile i; the epilogue (exp2 + reciprocal per sigmoid on the
// special-function unit) is the longer of the two, which is why it gets sixteen warps (four per
// scheduler), each reading its 64 columns 16 at a time.
//
// Every mbarrier wait is bounded: when a wait runs out the CTA records it in the status word,
// stops issuing work, drains what it has in flight and exits with its TMEM released.
#include "gsa_common.cuh"
#include "gsa_tc.cuh"

namespace gsa {

namespace {

constexpr int kTileKeys = 128;
constexpr int kNCols = 256;            // N of one MMA = (queries x heads) of a group
constexpr int kStages = 6;
constexpr int kEpiWarps = 16;          // 4 per scheduler: keeps the special-function unit fed
constexpr int kThreads = 64 + kEpiWarps * 32;
constexpr int kColsPerWarp = kNCols / (kEpiWarps / 4);   // accumulator columns one epilogue warp handles
constexpr int kChunkCols = 16;         // columns per tcgen05.ld

struct TcArgs {
    const float* w;
    const float* bI;
    float* scores;
    int64_t row_stride;
    int32_t* dev_status;
    RowRange rr;
    int32_t Lq, Lk;
    int32_t groups_per_batch;
    int32_t tiles_per_cta;
    long long wait_cycles;         // limit of every bounded wait
    int32_t withhold_q;            // fault injection: the q^I copy is left out, so its barrier is never completed
};

template <int DI>
struct SmemPlan {
    static constexpr int Q_BYTES = kNCols * DI * 2;
    static constexpr int K_BYTES = kTileKeys * DI * 2;
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + Q_BYTES;
    static constexpr int OFF_W = OFF_K + kStages * K_BYTES;
    static constexpr int OFF_B = OFF_W + kNCols * 4;
    static constexpr int OFF_BAR = OFF_B + 64;                    // 8-byte aligned
    static constexpr int N_BARS = 2 * kStages + 1 + 4 + 1;
    static constexpr int OFF_TMEM = OFF_BAR + N_BARS * 8;
    static constexpr int OFF_ABORT = OFF_TMEM + 8;
    static constexpr int TOTAL = OFF_ABORT + 8;
    static constexpr int ALLOC = TOTAL + 1024;                    // slack to align the base to 1024
};

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// sum_j w_j * sigmoid(x_j + b_j) over HI heads, with one reciprocal per group of up to four heads:
//   w1/a1 + w2/a2 = (w1 a2 + w2 a1) / (a1 a2),   a_j = 1 + 2^(-(x_j + b_j) log2 e).
// The exponent is clamped at 28 (sigmoid < 4e-9 there), so a product of four a_j stays below
// 2^116 and cannot overflow.  nb[j] = -b_j log2 e.
// The epilogue is bound by instruction issue, so for four and eight heads the arithmetic runs on the
// packed fp32 instructions of sm_100 (two values per instruction).  Adjacent heads (2i, 2i+1) share a
// register pair; the tree combines head 2i with 2i+2 and 2i+1 with 2i+3 (elementwise on the pairs), then,
// for eight heads, those with their counterparts four heads on: the even and the odd heads end up as one
// quotient each (four factors per denominator), and one more step joins the two under a single reciprocal:
// the special-function unit, which bounds this kernel, then sees nine operations per eight sigmoids.  To keep
// a product of eight factors inside fp32, the a_j of eight heads are carried scaled by 2^-12 (the offset
// rides in the exponent's bias term and in the added constant; exponent clamped at 27: sigmoid < 8e-9), so
// each lies in [2^-12, 2^15], the product of eight in [2^-96, 2^120] and a head's numerator term within
// w_j 2^-96 .. 2^96: nothing overflows and only weights below 2^-30 could be flushed.  The 2^-12 left over
// per quotient is folded into the weights, which the caller passes pre-scaled (kWeightScale).
// 37 issue slots per eight sigmoids instead of 54.
// RELU: sum_j w_j * max(x_j + b_j, 0) (Eq. 3), nb[j] = b_j; no special-function work at all.
template <int HI> constexpr float kOne = HI == 8 ? 2.44140625e-04f : 1.0f;             // 2^-12 : 1
template <int HI> constexpr float kExpClamp = HI == 8 ? 15.0f : 28.0f;                 // 27 - 12 : 28
template <int HI> constexpr float kExpBias = HI == 8 ? -12.0f : 0.0f;                  // added to nb[j] by the caller
template <int HI> constexpr float kWeightScale = HI == 8 ? 2.44140625e-04f : 1.0f;     // applied to w[j] by the caller

template <int HI, bool RELU>
__device__ __forceinline__ float gated_head_sum(const uint32_t* x, const float* w, const float (&nb)[HI]) {
    if constexpr (RELU) {
        float acc = 0.f;
#pragma unroll
        for (int j = 0; j < HI; ++j) acc = fmaf(w[j], fmaxf(__uint_as_float(x[j]) + nb[j], 0.f), acc);
        return acc;
    }
    if constexpr (HI >= 4) {
        constexpr int NP = HI / 2;
        const float2 kScale = make_float2(-1.4426950408889634f, -1.4426950408889634f), kOne2 = make_float2(kOne<HI>, kOne<HI>);
        float2 a2[NP];
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            const float2 y = __ffma2_rn(make_float2(__uint_as_float(x[2 * i]), __uint_as_float(x[2 * i + 1])), kScale,
                                        make_float2(nb[2 * i], nb[2 * i + 1]));
            a2[i] = __fadd2_rn(make_float2(ex2_approx(fminf(y.x, kExpClamp<HI>)), ex2_approx(fminf(y.y, kExpClamp<HI>))), kOne2);
        }
        // heads (0,1) with (2,3) [and (4,5) with (6,7)]: numerators and denominators of the pairs (0,2), (1,3)
        float2 n2[NP / 2], d2[NP / 2];
#pragma unroll
        for (int q = 0; q < NP / 2; ++q) {
            const float2 wp = make_float2(w[4 * q], w[4 * q + 1]), wq = make_float2(w[4 * q + 2], w[4 * q + 3]);
            n2[q] = __ffma2_rn(wp, a2[2 * q + 1], __fmul2_rn(wq, a2[2 * q]));
            d2[q] = __fmul2_rn(a2[2 * q], a2[2 * q + 1]);
        }
        if constexpr (HI == 8) {
            const float2 nc = __ffma2_rn(n2[0], d2[1], __fmul2_rn(n2[1], d2[0]));     // even heads | odd heads
            const float2 dc = __fmul2_rn(d2[0], d2[1]);
            return fmaf(nc.x, dc.y, nc.y * dc.x) * rcp_approx(dc.x * dc.y);
        } else {
            return fmaf(n2[0].x, d2[0].y, n2[0].y * d2[0].x) * rcp_approx(d2[0].x * d2[0].y);
        }
    } else {
        float a[HI];
#pragma unroll
        for (int j = 0; j < HI; ++j)
            a[j] = 1.0f + ex2_approx(fminf(fmaf(__uint_as_float(x[j]), -1.4426950408889634f, nb[j]), 28.0f));
        if constexpr (HI == 2) return fmaf(w[0], a[1], w[1] * a[0]) * rcp_approx(a[0] * a[1]);
        else return w[0] * rcp_approx(a[0]);
    }
}

// instruction descriptor: D fp32, A = B = bf16, both K-major, M = 128, N = 256
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kNCols >> 3) << 17) |
                            ((uint32_t)(kTileKeys >> 4) << 24);

template <int DI, int HI, bool RELU>
__global__ void __launch_bounds__(kThreads, 1)
gsa_indexer_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q,
                      const TcArgs a) {
    using P = SmemPlan<DI>;
    constexpr int NQ = kNCols / HI;             // queries per group
    constexpr int KSTEPS = DI / 16;
    constexpr int ROW_BYTES = DI * 2;

    // ---- which work is mine ------------------------------------------------------------------
    const int g = (int)gridDim.y - 1 - (int)blockIdx.y;               // heavy (late) groups first
    const int bl = g / a.groups_per_batch;
    const int tr0 = (g % a.groups_per_batch) * NQ;
    const int nq = min(NQ, a.rr.R - tr0);
    const int b = a.rr.b0 + bl;
    const int t0 = a.rr.q_begin + tr0;
    const int off = a.Lk - a.Lq;
    const int n_vis_last = off + t0 + nq;                             // visible keys of the group's last query
    const int tiles_group = (n_vis_last + kTileKeys - 1) / kTileKeys;
    const int tile0 = blockIdx.x * a.tiles_per_cta;
    const int ntiles = min(a.tiles_per_cta, tiles_group - tile0);
    if (ntiles <= 0) return;                                          // whole CTA, before any barrier
    {   // an earlier CTA gave up: leave, all threads together (one thread reads the word)
        __shared__ int s_go;
        if (threadIdx.x == 0) s_go = *reinterpret_cast<volatile int32_t*>(a.dev_status) == kDevOk;
        __syncthreads();
        if (!s_go) return;
    }

    extern __shared__ unsigned char dyn_smem_raw[];
    const uint32_t raw_u32 = smem_u32(dyn_smem_raw);
    const uint32_t pad = (1024u - (raw_u32 & 1023u)) & 1023u;
    unsigned char* smem = dyn_smem_raw + pad;
    const uint32_t sbase = raw_u32 + pad;

    float* s_w = reinterpret_cast<float*>(smem + P::OFF_W);
    float* s_b = reinterpret_cast<float*>(smem + P::OFF_B);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + P::OFF_TMEM);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + P::OFF_ABORT);
    const uint32_t bar0 = sbase + P::OFF_BAR;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_empty = [&](int s) { return bar0 + 8u * (kStages + s); };
    const uint32_t bar_q = bar0 + 8u * (2 * kStages);
    auto bar_tfull = [&](int i) { return bar0 + 8u * (2 * kStages + 1 + i); };
    auto bar_tempty = [&](int i) { return bar0 + 8u * (2 * kStages + 3 + i); };
    const uint32_t bar_drain = bar0 + 8u * (2 * kStages + 5);         // give-up path only

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        mbar_init(bar_q, 1);
        for (int i = 0; i < 2; ++i) { mbar_init(bar_tfull(i), 1); mbar_init(bar_tempty(i), kEpiWarps); }
        mbar_init(bar_drain, 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(sbase + P::OFF_TMEM)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (warp >= 2) {
        const int e = threadIdx.x - 64;                               // 0..255 = (query, head) column
        if (e < kNCols) {
            const int qi = e / HI, j = e % HI;
            // (sigmoid path with eight heads: weights pre-scaled by the power of two the head sum leaves over)
            s_w[e] = qi < nq ? a.w[((size_t)b * a.Lq + t0 + qi) * HI + j] * (RELU ? 1.0f : kWeightScale<HI>) : 0.f;
            if (e < 8) s_b[e] = (a.bI && e < HI) ? a.bI[e] : 0.f;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *s_tmem;
    // what this thread has put in flight (the copy producer's and the MMA issuer's own counts)
    int copies_issued = 0, mma_tiles_issued = 0;
    bool q_issued = false;

    if (warp == 0) {
        // ================= TMA producer =======================================================
        if (lane == 0) {
            if (!a.withhold_q) {
                mbar_expect_tx(bar_q, P::Q_BYTES);
                tma_load_2d(sbase + P::OFF_Q, &tm_q, 0, (b * a.Lq + t0) * HI, bar_q);
                q_issued = true;
            }
            for (int i = 0; i < ntiles && !*s_abort; ++i) {
                const int s = i % kStages;
                if (!mbar_wait(bar_empty(s), ((i / kStages) & 1) ^ 1, s_abort, a.wait_cycles)) break;
                mbar_expect_tx(bar_full(s), P::K_BYTES);
                tma_load_2d(sbase + P::OFF_K + s * P::K_BYTES, &tm_k, 0, b * a.Lk + (tile0 + i) * kTileKeys,
                            bar_full(s));
                copies_issued = i + 1;
            }
            if (copies_issued < ntiles) atomicCAS(a.dev_status, kDevOk, kDevTimeoutTma);
        }
    } else if (warp == 1) {
        // ================= MMA issuer =========================================================
        if (lane == 0) {
            bool ok = mbar_wait(bar_q, 0, s_abort, a.wait_cycles);
            const uint64_t bdesc = make_kmajor_desc<ROW_BYTES>(sbase + P::OFF_Q);
            for (int i = 0; ok && i < ntiles; ++i) {
                const int s = i % kStages, buf = i & 1;
                if (!mbar_wait(bar_tempty(buf), ((i >> 1) & 1) ^ 1, s_abort, a.wait_cycles)) { ok = false; break; }
                if (!mbar_wait(bar_full(s), (i / kStages) & 1, s_abort, a.wait_cycles)) { ok = false; break; }
                tc_fence_after();
                const uint64_t adesc = make_kmajor_desc<ROW_BYTES>(sbase + P::OFF_K + s * P::K_BYTES);
#pragma unroll
                for (int k = 0; k < KSTEPS; ++k)           // 16 K-elements = 32 bytes = 2 descriptor units
                    tc_mma_bf16(tmem_base + buf * kNCols, adesc + 2 * k, bdesc + 2 * k, kIdesc, k > 0);
                tc_commit(bar_empty(s));                   // stage reusable once these MMAs have read it
                tc_commit(bar_tfull(buf));                 // accumulator ready for the epilogue
                mma_tiles_issued = i + 1;
            }
            if (!ok) atomicCAS(a.dev_status, kDevOk, kDevTimeoutMma);
        }
    } else {
        // ================= epilogue: sigmoid, head weights, head sum, store ===================
        const int ew = warp - 2;
        const int quad = warp & 3;                          // TMEM lanes this warp may touch: 32*quad ..
        const int part = ew >> 2;                           // which kColsPerWarp of the 256 columns
        constexpr int QPC = kChunkCols / HI;                // queries per 16-column chunk
        constexpr int NCHUNK = kColsPerWarp / kChunkCols;
        float bias[HI];
#pragma unroll
        for (int j = 0; j < HI; ++j) bias[j] = RELU ? s_b[j] : fmaf(s_b[j], -1.4426950408889634f, kExpBias<HI>);
        for (int i = 0; i < ntiles; ++i) {
            const int buf = i & 1;
            if (!mbar_wait(bar_tfull(buf), (i >> 1) & 1, s_abort, a.wait_cycles)) {
                if (lane == 0) atomicCAS(a.dev_status, kDevOk, kDevTimeoutEpi);
                break;
            }
            tc_fence_after();
            const int s = (tile0 + i) * kTileKeys + quad * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * kNCols + part * kColsPerWarp;
            // columns are read 16 at a time, the next chunk's load in flight behind the current
            // chunk's arithmetic
            float* const out_col = a.scores + ((int64_t)bl * a.rr.R + tr0) * a.row_stride + s;
            auto do_chunk = [&](const uint32_t (&r)[kChunkCols], int c) {
                const int q_first = (part * kColsPerWarp + c * kChunkCols) / HI;
#pragma unroll
                for (int qq = 0; qq < QPC; ++qq) {
                    const int qi = q_first + qq;
                    float wv[HI];
                    if constexpr (HI >= 4) {
#pragma unroll
                        for (int j = 0; j < HI; j += 4) {
                            const float4 v = *reinterpret_cast<const float4*>(s_w + qi * HI + j);
                            wv[j] = v.x; wv[j + 1] = v.y; wv[j + 2] = v.z; wv[j + 3] = v.w;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < HI; ++j) wv[j] = s_w[qi * HI + j];
                    }
                    const float acc = gated_head_sum<HI, RELU>(&r[qq * HI], wv, bias);
                    if (qi < nq && s <= off + t0 + qi) out_col[(int64_t)qi * a.row_stride] = acc;
                }
            };
            uint32_t ra[kChunkCols], rb[kChunkCols];
            tc_ld16(taddr, ra);
#pragma unroll
            for (int c = 0; c < NCHUNK; c += 2) {
                tc_wait_ld16(ra);
                tc_ld16(taddr + (c + 1) * kChunkCols, rb);
                do_chunk(ra, c);
                tc_wait_ld16(rb);
                if (c + 2 < NCHUNK) tc_ld16(taddr + (c + 2) * kChunkCols, ra);
                do_chunk(rb, c + 1);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty(buf));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*s_abort) {
        // Give-up path.  Every role has left its loop, but what was issued before is still under way: copies
        // land in this CTA's stages, MMAs read them and write its TMEM, commits arrive on its barriers.  None
        // of that may outlive the CTA, whose TMEM and shared memory go to the next one.  All of it completes by
        // itself (nothing issued waits for anything that was not), so these polls end; each is bounded anyway.
        if (warp == 0 && lane == 0) {
            if (q_issued) mbar_drain(bar_q, 0);
            for (int i = max(0, copies_issued - kStages); i < copies_issued; ++i)
                mbar_drain(bar_full(i % kStages), (i / kStages) & 1);
        }
        if (warp == 1 && lane == 0) {
            tc_commit(bar_drain);                          // arrives once every MMA issued so far has completed
            mbar_drain(bar_drain, 0);
            for (int i = max(0, mma_tiles_issued - kStages); i < mma_tiles_issued; ++i)
                mbar_drain(bar_empty(i % kStages), (i / kStages) & 1);
            for (int i = max(0, mma_tiles_issued - 2); i < mma_tiles_issued; ++i)
                mbar_drain(bar_tfull(i & 1), (i >> 1) & 1);
        }
        tc_fence_before();
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

template <int DI, int HI, bool RELU>
cudaError_t launch_t(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* qI, const __nv_bfloat16* kI,
                     const float* w, const float* bI, float* scores, int64_t row_stride, int32_t* dev_status,
                     cudaStream_t st) {
    using P = SmemPlan<DI>;
    constexpr int NQ = kNCols / HI;
    CUtensorMap tm_k, tm_q;
    if (!make_rows_tmap(&tm_k, kI, (uint64_t)p.B * p.Lk, DI, kTileKeys)) return cudaErrorUnknown;
    if (!make_rows_tmap(&tm_q, qI, (uint64_t)p.B * p.Lq * HI, DI, kNCols)) return cudaErrorUnknown;

    TcArgs a;
    a.w = w; a.bI = bI; a.scores = scores; a.row_stride = row_stride; a.dev_status = dev_status;
    a.rr = rr; a.Lq = p.Lq; a.Lk = p.Lk;
    a.groups_per_batch = (rr.R + NQ - 1) / NQ;
    const int groups = rr.nb * a.groups_per_batch;
    const int n_vis_max = p.Lk - p.Lq + rr.q_begin + rr.R;
    const int tiles_max = (n_vis_max + kTileKeys - 1) / kTileKeys;
    // enough CTAs to fill the GPU a few times over, but runs long enough to amortise the q^I load
    int64_t total_tiles = (int64_t)groups * tiles_max;
    int tpc = (int)(total_tiles / (sm_count() * 4));
    tpc = tpc < 4 ? 4 : (tpc > 64 ? 64 : tpc);
    a.tiles_per_cta = tpc;
    a.wait_cycles = wait_limit_cycles();
    a.withhold_q = withhold_first_copy() ? 1 : 0;
    dim3 grid((tiles_max + tpc - 1) / tpc, groups);

    // one CTA per SM: the kernel allocates all 512 TMEM columns, so a second resident CTA would
    // only sit in tcgen05.alloc until the first one leaves
    constexpr int kSmem = P::ALLOC > 120 * 1024 ? P::ALLOC : 120 * 1024;
    auto kern = gsa_indexer_tc_kernel<DI, HI, RELU>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, kSmem, st>>>(tm_k, tm_q, a);
    ++g_launches;
    return cudaGetLastError();
}

}  // namespace

bool indexer_tc_supported(const gsa_params_t& p) {
    if (!(p.dI == 64 || p.dI == 32)) return false;
    if (!(p.HI == 1 || p.HI == 2 || p.HI == 4 || p.HI == 8)) return false;
    if ((int64_t)p.B * p.Lq * p.HI >= (1ll << 31) || (int64_t)p.B * p.Lk >= (1ll << 31)) return false;
    return get_encode_fn() != nullptr;
}

cudaError_t launch_indexer_tc(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* qI,
                              const __nv_bfloat16* kI, const float* w, const float* bI, float* scores,
                              int64_t row_stride, int32_t* dev_status, cudaStream_t st) {
    if (rr.rows() <= 0) return cudaSuccess;
#define GSA_TC_CASE(DI_, HI_) \
    if (p.dI == DI_ && p.HI == HI_) \
        return p.act == 1 ? launch_t<DI_, HI_, true>(p, rr, qI, kI, w, bI, scores, row_stride, dev_status, st) \
                          : launch_t<DI_, HI_, false>(p, rr, qI, kI, w, bI, scores, row_stride, dev_status, st)
    GSA_TC_CASE(64, 8); GSA_TC_CASE(64, 4); GSA_TC_CASE(64, 2); GSA_TC_CASE(64, 1);
    GSA_TC_CASE(32, 8); GSA_TC_CASE(32, 4); GSA_TC_CASE(32, 2); GSA_TC_CASE(32, 1);
#undef GSA_TC_CASE
    return cudaErrorInvalidValue;
}

}  // namespace gsa
