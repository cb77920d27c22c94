// Upstream projections of a GSA layer (text below Eq. 7; Eq. 9; Eq. 10) as ONE dense GEMM on the
// 5th-generation tensor cores, with the output routing and the head-weight sigmoid in the epilogue:
//
//     C[token, n] = sum_c H[token, c] * Wt[n, c]            tcgen05.mma, bf16 x bf16 -> fp32 in TMEM
//     columns n:  q^I (H^I*d^I) | k^I (d^I) | head weights (8, the first H^I used) | g1 logits | g2 logits
//     q^I, k^I, g1, g2 are rounded to bf16 once; head weights leave as fp32 sigmoid(C).
//
// A persistent CTA walks output tiles of 128 tokens x 256 columns.  Warp 0 feeds a ring of shared-
// memory stages by TMA (a 128 x 64 block of H and a 256 x 64 block of Wt per stage, 128-byte
// swizzle), warp 1 issues the MMAs (four k-steps per stage) and owns the TMEM allocation, warps
// 2..9 are the epilogue.  Two 256-column accumulators alternate, so the MMAs of the next tile run
// while the epilogue converts and stores the current one.  Rows and columns of a tile that fall
// outside the matrices are zero-filled by TMA and masked at the store.
//
// Every mbarrier wait is bounded: when one runs out the CTA records it in the status word, stops
// issuing work, drains what it has in flight and exits with its TMEM released.
#include "gsa_common.cuh"
#include "gsa_tc.cuh"

namespace gsa {

namespace {

constexpr int kTileM = 128;
constexpr int kTileN = 256;
constexpr int kBlockK = 64;
constexpr int kPStages = 4;
constexpr int kPEpiWarps = 8;
constexpr int kPThreads = 64 + kPEpiWarps * 32;
constexpr int kA_BYTES = kTileM * kBlockK * 2;          // 16 KB
constexpr int kB_BYTES = kTileN * kBlockK * 2;          // 32 KB
constexpr int kStageBytes = kA_BYTES + kB_BYTES;
constexpr int kOffBar = kPStages * kStageBytes;
constexpr int kNBars = 2 * kPStages + 4 + 1;
constexpr int kOffTmem = kOffBar + kNBars * 8;
constexpr int kOffAbort = kOffTmem + 8;
constexpr int kSmemTotal = kOffAbort + 8 + 1024;        // slack to align the base to 1024
constexpr uint32_t kIdescP = make_idesc_bf16(kTileM, kTileN);

struct ProjArgs {
    __nv_bfloat16* qI;
    __nv_bfloat16* kI;
    float* w;
    __nv_bfloat16* g1;
    __nv_bfloat16* g2;
    int32_t* dev_status;
    int32_t M, K, N;               // tokens, d_model, stacked output columns
    int32_t n_q, n_k, HI, n_g1, n_g2;
    int32_t m_tiles, n_tiles;
    long long wait_cycles;         // limit of every bounded wait
    int32_t withhold_first;        // fault injection: the first stage's copies are left out (its barrier is never completed)
};

__global__ void __launch_bounds__(kPThreads, 1)
gsa_project_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_w,
                   const ProjArgs a) {
    {   // an earlier CTA or launch gave up: leave, all threads together (one thread reads the word)
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
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + kOffTmem);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + kOffAbort);
    const uint32_t bar0 = sbase + kOffBar;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_empty = [&](int s) { return bar0 + 8u * (kPStages + s); };
    auto bar_tfull = [&](int i) { return bar0 + 8u * (2 * kPStages + i); };
    auto bar_tempty = [&](int i) { return bar0 + 8u * (2 * kPStages + 2 + i); };
    const uint32_t bar_drain = bar0 + 8u * (2 * kPStages + 4);        // give-up path only

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kPStages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar_tfull(i), 1); mbar_init(bar_tempty(i), kPEpiWarps); }
        mbar_init(bar_drain, 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(sbase + kOffTmem) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *s_tmem;

    const int n_tiles_total = a.m_tiles * a.n_tiles;
    const int kblocks = (a.K + kBlockK - 1) / kBlockK;
    // what this thread has put in flight (the copy producer's and the MMA issuer's own counts)
    uint32_t copies_issued = 0;                            // stages filled so far (all tiles)
    uint32_t mma_blocks_issued = 0, mma_tiles_committed = 0;
    bool first_withheld = false;

    if (warp == 0) {
        // ================= TMA producer =======================================================
        if (lane == 0) {
            bool gave_up = false;
            for (int tile = blockIdx.x; tile < n_tiles_total && !gave_up && !*s_abort; tile += gridDim.x) {
                const int m0 = (tile / a.n_tiles) * kTileM, n0 = (tile % a.n_tiles) * kTileN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    const uint32_t it = copies_issued;
                    const int s = it % kPStages;
                    if (!mbar_wait(bar_empty(s), ((it / kPStages) & 1) ^ 1, s_abort, a.wait_cycles)) { gave_up = true; break; }
                    if (it == 0 && a.withhold_first) {
                        first_withheld = true;             // (counted as issued; the give-up path skips it)
                    } else {
                        mbar_expect_tx(bar_full(s), kStageBytes);
                        const uint32_t dst = sbase + s * kStageBytes;
                        tma_load_2d(dst, &tm_h, kb * kBlockK, m0, bar_full(s));
                        tma_load_2d(dst + kA_BYTES, &tm_w, kb * kBlockK, n0, bar_full(s));
                    }
                    copies_issued = it + 1;
                }
            }
            if (gave_up) atomicCAS(a.dev_status, kDevOk, kDevTimeoutTma);
        }
    } else if (warp == 1) {
        // ================= MMA issuer =========================================================
        if (lane == 0) {
            uint32_t it = 0, tl = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < n_tiles_total; tile += gridDim.x, ++tl) {
                const int buf = tl & 1;
                if (!mbar_wait(bar_tempty(buf), ((tl >> 1) & 1) ^ 1, s_abort, a.wait_cycles)) { ok = false; break; }
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % kPStages;
                    if (!mbar_wait(bar_full(s), (it / kPStages) & 1, s_abort, a.wait_cycles)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t adesc = make_kmajor_desc<128>(sbase + s * kStageBytes);
                    const uint64_t bdesc = make_kmajor_desc<128>(sbase + s * kStageBytes + kA_BYTES);
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k)      // 16 K-elements = 32 bytes = 2 descriptor units
                        tc_mma_bf16(tmem_base + buf * kTileN, adesc + 2 * k, bdesc + 2 * k, kIdescP, (kb | k) != 0);
                    tc_commit(bar_empty(s));                    // stage reusable once these MMAs have read it
                    mma_blocks_issued = it + 1;
                }
                if (ok) {
                    tc_commit(bar_tfull(buf));                  // accumulator ready for the epilogue
                    mma_tiles_committed = tl + 1;
                }
            }
            if (!ok) atomicCAS(a.dev_status, kDevOk, kDevTimeoutMma);
        }
    } else {
        // ================= epilogue: route, round / sigmoid, store =============================
        const int ew = warp - 2;
        const int quad = warp & 3;                          // TMEM lanes this warp may touch: 32*quad ..
        const int half = ew >> 2;                           // which 128 of the tile's 256 columns
        const int o_k = a.n_q, o_w = o_k + a.n_k, o_g1 = o_w + 8, o_g2 = o_g1 + a.n_g1;
        uint32_t tl = 0;
        for (int tile = blockIdx.x; tile < n_tiles_total; tile += gridDim.x, ++tl) {
            const int buf = tl & 1;
            if (!mbar_wait(bar_tfull(buf), (tl >> 1) & 1, s_abort, a.wait_cycles)) {
                if (lane == 0) atomicCAS(a.dev_status, kDevOk, kDevTimeoutEpi);
                break;
            }
            tc_fence_after();
            const int m = (tile / a.n_tiles) * kTileM + quad * 32 + lane;       // this thread's token
            const int n_base = (tile % a.n_tiles) * kTileN + half * 128;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * kTileN + half * 128;
            auto store8 = [&](const uint32_t* r, int n8) {   // 8 consecutive columns starting at n8 (a multiple of 8)
                if (m >= a.M || n8 >= a.N) return;
                if (n8 >= o_w && n8 < o_g1) {                // head weights: fp32 sigmoid
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j < a.HI) a.w[(size_t)m * a.HI + j] = fast_sigmoid(__uint_as_float(r[j]));
                    return;
                }
                __nv_bfloat16* dst;
                if (n8 < o_k)        dst = a.qI + (size_t)m * a.n_q + n8;
                else if (n8 < o_w)   dst = a.kI + (size_t)m * a.n_k + (n8 - o_k);
                else if (n8 < o_g2)  dst = a.g1 + (size_t)m * a.n_g1 + (n8 - o_g1);
                else                 dst = a.g2 + (size_t)m * a.n_g2 + (n8 - o_g2);
                uint4 v;
                v.x = pack_bf16(__uint_as_float(r[0]), __uint_as_float(r[1]));
                v.y = pack_bf16(__uint_as_float(r[2]), __uint_as_float(r[3]));
                v.z = pack_bf16(__uint_as_float(r[4]), __uint_as_float(r[5]));
                v.w = pack_bf16(__uint_as_float(r[6]), __uint_as_float(r[7]));
                *reinterpret_cast<uint4*>(dst) = v;
            };
            uint32_t ra[16], rb[16];
            tc_ld16(taddr, ra);
#pragma unroll
            for (int c = 0; c < 8; c += 2) {
                tc_wait_ld16(ra);
                tc_ld16(taddr + (c + 1) * 16, rb);
                store8(ra, n_base + c * 16);
                store8(ra + 8, n_base + c * 16 + 8);
                tc_wait_ld16(rb);
                if (c + 2 < 8) tc_ld16(taddr + (c + 2) * 16, ra);
                store8(rb, n_base + (c + 1) * 16);
                store8(rb + 8, n_base + (c + 1) * 16 + 8);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty(buf));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*s_abort) {
        // Give-up path: what was issued before a wait ran out is still under way (copies into this CTA's
        // stages, MMAs that read them and write its TMEM, commits onto its barriers) and must not outlive the
        // CTA.  All of it completes by itself, so these polls end; each is bounded anyway.
        if (warp == 0 && lane == 0) {
            const uint32_t back = copies_issued < (uint32_t)kPStages ? copies_issued : (uint32_t)kPStages;
            for (uint32_t i = 0; i < back; ++i) {
                const uint32_t f = copies_issued - 1 - i;
                if (f == 0 && first_withheld) continue;    // never issued
                mbar_drain(bar_full(f % kPStages), (f / kPStages) & 1);
            }
        }
        if (warp == 1 && lane == 0) {
            tc_commit(bar_drain);                          // arrives once every MMA issued so far has completed
            mbar_drain(bar_drain, 0);
            const uint32_t back = mma_blocks_issued < (uint32_t)kPStages ? mma_blocks_issued : (uint32_t)kPStages;
            for (uint32_t i = 0; i < back; ++i) {
                const uint32_t f = mma_blocks_issued - 1 - i;
                mbar_drain(bar_empty(f % kPStages), (f / kPStages) & 1);
            }
            for (uint32_t i = 0; i < 2 && i < mma_tiles_committed; ++i) {
                const uint32_t f = mma_tiles_committed - 1 - i;
                mbar_drain(bar_tfull(f & 1), (f >> 1) & 1);
            }
        }
        tc_fence_before();
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

}  // namespace

int project_columns(const gsa_params_t& p) {
    return p.HI * p.dI + p.dI + 8 + p.n_h * p.d_h + p.n_kv * p.d_h;
}

cudaError_t launch_project(const gsa_params_t& p, int d_model, const __nv_bfloat16* H, const __nv_bfloat16* Wt,
                           __nv_bfloat16* qI, __nv_bfloat16* kI, float* w, __nv_bfloat16* g1, __nv_bfloat16* g2,
                           int32_t* dev_status, cudaStream_t st) {
    ProjArgs a;
    a.qI = qI; a.kI = kI; a.w = w; a.g1 = g1; a.g2 = g2; a.dev_status = dev_status;
    a.M = p.B * p.Lk; a.K = d_model; a.N = project_columns(p);
    a.n_q = p.HI * p.dI; a.n_k = p.dI; a.HI = p.HI; a.n_g1 = p.n_h * p.d_h; a.n_g2 = p.n_kv * p.d_h;
    a.m_tiles = (a.M + kTileM - 1) / kTileM;
    a.n_tiles = (a.N + kTileN - 1) / kTileN;
    a.wait_cycles = wait_limit_cycles();
    a.withhold_first = withhold_first_copy() ? 1 : 0;
    CUtensorMap tm_h, tm_w;
    if (!make_kblock_tmap(&tm_h, H, (uint64_t)a.M, (uint64_t)a.K, kTileM)) return cudaErrorUnknown;
    if (!make_kblock_tmap(&tm_w, Wt, (uint64_t)a.N, (uint64_t)a.K, kTileN)) return cudaErrorUnknown;
    cudaError_t e = cudaFuncSetAttribute(gsa_project_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTotal);
    if (e != cudaSuccess) return e;
    const int sms = sm_count();
    const int tiles = a.m_tiles * a.n_tiles;
    gsa_project_kernel<<<tiles < sms ? tiles : sms, kPThreads, kSmemTotal, st>>>(tm_h, tm_w, a);
    ++g_launches;
    return cudaGetLastError();
}


// C[M, N] = A[M, K] * Bt[N, K]^T, bf16 in, fp32 accumulate, bf16 out: the same kernel with a single
// output block (used for the output projection W_O).
cudaError_t launch_gemm_bf16(int M, int K, int N, const __nv_bfloat16* A, const __nv_bfloat16* Bt, __nv_bfloat16* C,
                             int32_t* dev_status, cudaStream_t st) {
    ProjArgs a;
    a.qI = C; a.kI = nullptr; a.w = nullptr; a.g1 = nullptr; a.g2 = nullptr; a.dev_status = dev_status;
    a.M = M; a.K = K; a.N = N;
    a.n_q = N; a.n_k = 0; a.HI = 0; a.n_g1 = 0; a.n_g2 = 0;
    a.m_tiles = (M + kTileM - 1) / kTileM;
    a.n_tiles = (N + kTileN - 1) / kTileN;
    a.wait_cycles = wait_limit_cycles();
    a.withhold_first = withhold_first_copy() ? 1 : 0;
    CUtensorMap tm_a, tm_b;
    if (!make_kblock_tmap(&tm_a, A, (uint64_t)M, (uint64_t)K, kTileM)) return cudaErrorUnknown;
    if (!make_kblock_tmap(&tm_b, Bt, (uint64_t)N, (uint64_t)K, kTileN)) return cudaErrorUnknown;
    cudaError_t e = cudaFuncSetAttribute(gsa_project_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTotal);
    if (e != cudaSuccess) return e;
    const int sms = sm_count();
    const int tiles = a.m_tiles * a.n_tiles;
    gsa_project_kernel<<<tiles < sms ? tiles : sms, kPThreads, kSmemTotal, st>>>(tm_a, tm_b, a);
    ++g_launches;
    return cudaGetLastError();
}

}  // namespace gsa
