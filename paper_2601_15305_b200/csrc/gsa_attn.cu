// Sparse gated attention (Eq. 9, 11, 12, 10): one warp per (query, KV head).
//
// The warp gathers the selected keys' K and V' rows of its KV head (d_h bf16 = 16-byte chunks,
// cp.async, L2-only) into a private multi-stage ring in shared memory, 16 keys per stage, and
// runs an online-softmax loop on bf16 tensor-core MMAs (m16n8k16, fp32 accumulate):
//     S[head, key]  = Q[head, :] . K[key, :]        rows = the G query heads of the KV group
//     O[head, :]   += P[head, key] * V'[key, :]
// The eight warps of a CTA cover the eight KV heads of one query, so together they fetch each
// selected token's whole 2 KB K row and 2 KB V' row exactly once.  G2 is either applied by a
// streaming pre-pass (V' = bf16(V * sigmoid(g2)), prefill) or inside the gather (decode, where
// gating the whole cache would cost more than the attention); G1 is applied to the fp32
// accumulator before the single rounding to bf16.
#include "gsa_common.cuh"

namespace gsa {

namespace {

constexpr int kTileKeys = 16;

struct AttnArgs {
    const __nv_bfloat16* Q;
    const __nv_bfloat16* K;
    const __nv_bfloat16* V;
    const __nv_bfloat16* g1;
    const __nv_bfloat16* g2;
    const int32_t* idx;
    const int32_t* kt;
    __nv_bfloat16* out;
    RowRange rr;
    IdxLayout il;
    int32_t Lq, Lk, n_h, n_kv, k_max;
    int32_t q_per_cta;
    float scale_log2;     // sm_scale * log2(e)
};

template <int DH, int G, bool FUSE_G2, int STAGES>
__global__ void __launch_bounds__(256) gsa_sparse_attn_kernel(const AttnArgs a) {
    constexpr int ROW_BYTES = DH * 2;
    constexpr int CHUNKS = ROW_BYTES / 16;                  // 16-byte chunks per row: 8 or 16
    constexpr int TENSORS = FUSE_G2 ? 3 : 2;
    constexpr int TILE_BYTES = kTileKeys * ROW_BYTES;       // one tensor, one stage
    constexpr int STAGE_BYTES = TENSORS * TILE_BYTES;
    constexpr int KSTEPS = DH / 16;                         // QK^T k-steps
    constexpr int NT_O = DH / 8;                            // output n-tiles
    constexpr int ROWS_PER_IT = 32 / CHUNKS;                // key rows one warp-wide cp.async covers
    constexpr int ITS = kTileKeys / ROWS_PER_IT;

    extern __shared__ __align__(128) unsigned char smem[];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int slot = wid / a.n_kv, g = wid % a.n_kv;
    const int lr = blockIdx.x * a.q_per_cta + slot;
    if (slot >= a.q_per_cta || lr >= a.rr.rows()) return;   // warp-uniform; no CTA barriers below
    const int b = a.rr.b0 + lr / a.rr.R;
    const int t = a.rr.q_begin + lr % a.rr.R;
    const int64_t irow = a.il.row(b, t);
    const int32_t* __restrict__ idx_row = a.idx + irow * a.k_max;
    const int k_eff = a.kt[irow];

    unsigned char* my_smem = smem + (size_t)wid * STAGES * STAGE_BYTES;
    const uint32_t my_smem_u32 = smem_u32(my_smem);

    const int qrow = lane >> 2, qcol = (lane & 3) * 2;
    const bool real_row = qrow < G;
    const int h = g * G + (real_row ? qrow : 0);
    const size_t q_off = (((size_t)b * a.Lq + t) * a.n_h + h) * DH;

    // Q as the A operand: rows = heads of the group (rows >= G are zero padding)
    uint32_t qa[KSTEPS][2];
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ++ks) {
        qa[ks][0] = real_row ? *reinterpret_cast<const uint32_t*>(a.Q + q_off + ks * 16 + qcol) : 0u;
        qa[ks][1] = real_row ? *reinterpret_cast<const uint32_t*>(a.Q + q_off + ks * 16 + 8 + qcol) : 0u;
    }

    const size_t kv_batch = (size_t)b * a.Lk;
    const int my_chunk = lane % CHUNKS, my_sub = lane / CHUNKS;

    auto issue_tile = [&](int tile) {
        const int stage = tile % STAGES;
        const int j0 = tile * kTileKeys;
        int pos_l = 0;
        if (lane < kTileKeys) {
            const int j = j0 + lane;
            pos_l = idx_row[j < k_eff ? j : 0];           // padding keys re-read a valid row; P = 0 there
        }
        const uint32_t sbase = my_smem_u32 + stage * STAGE_BYTES;
#pragma unroll
        for (int it = 0; it < ITS; ++it) {
            const int r = it * ROWS_PER_IT + my_sub;
            const int pos = __shfl_sync(0xFFFFFFFFu, pos_l, r);
            const size_t goff = ((kv_batch + pos) * a.n_kv + g) * DH + my_chunk * 8;
            const uint32_t soff = r * ROW_BYTES + ((my_chunk ^ (r & 7)) << 4);
            cp_async16(sbase + soff, a.K + goff);
            cp_async16(sbase + TILE_BYTES + soff, a.V + goff);
            if (FUSE_G2) cp_async16(sbase + 2 * TILE_BYTES + soff, a.g2 + goff);
        }
    };

    float o_acc[NT_O][4];
#pragma unroll
    for (int i = 0; i < NT_O; ++i) { o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f; }
    float m_run = -INFINITY, l_run = 0.f;

    const int ntiles = (k_eff + kTileKeys - 1) / kTileKeys;
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < ntiles) issue_tile(s);
        cp_async_commit();
    }

    for (int tile = 0; tile < ntiles; ++tile) {
        if (tile + STAGES - 1 < ntiles) issue_tile(tile + STAGES - 1);
        cp_async_commit();
        cp_async_wait<STAGES - 1>();
        __syncwarp();
        const uint32_t sbase = my_smem_u32 + (tile % STAGES) * STAGE_BYTES;

        if (FUSE_G2) {       // Eq. 9 in place: V tile <- bf16(V * sigmoid(g2))
            unsigned char* sv = my_smem + (tile % STAGES) * STAGE_BYTES + TILE_BYTES;
            unsigned char* sg = sv + TILE_BYTES;
#pragma unroll
            for (int c = lane; c < kTileKeys * CHUNKS; c += 32) {
                uint4 vv = *reinterpret_cast<uint4*>(sv + c * 16);
                const uint4 gg = *reinterpret_cast<const uint4*>(sg + c * 16);
                __nv_bfloat162* v2 = reinterpret_cast<__nv_bfloat162*>(&vv);
                const __nv_bfloat162* g2v = reinterpret_cast<const __nv_bfloat162*>(&gg);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 vf = __bfloat1622float2(v2[e]), gf = __bfloat1622float2(g2v[e]);
                    v2[e] = __floats2bfloat162_rn(vf.x * fast_sigmoid(gf.x), vf.y * fast_sigmoid(gf.y));
                }
                *reinterpret_cast<uint4*>(sv + c * 16) = vv;
            }
            __syncwarp();
        }

        // ---- S = Q K^T over the 16 keys of the tile (two n-tiles of 8 keys) -----------------
        float s_acc[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            s_acc[nt][0] = s_acc[nt][1] = s_acc[nt][2] = s_acc[nt][3] = 0.f;
            const int key = nt * 8 + (lane & 7);
#pragma unroll
            for (int kk = 0; kk < KSTEPS / 2; ++kk) {
                const int chunk = kk * 4 + (lane >> 3);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(b0, b1, b2, b3, sbase + key * ROW_BYTES + ((chunk ^ (key & 7)) << 4));
                mma_bf16_16816(s_acc[nt], qa[2 * kk][0], 0u, qa[2 * kk][1], 0u, b0, b1);
                mma_bf16_16816(s_acc[nt], qa[2 * kk + 1][0], 0u, qa[2 * kk + 1][1], 0u, b2, b3);
            }
        }

        // ---- online softmax on row lane/4 ---------------------------------------------------
        const int j0 = tile * kTileKeys;
        float p[2][2];
        float tmax = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int j = j0 + nt * 8 + qcol + e;
                const float sv = j < k_eff ? s_acc[nt][e] * a.scale_log2 : -INFINITY;
                p[nt][e] = sv;
                tmax = fmaxf(tmax, sv);
            }
        tmax = fmaxf(tmax, __shfl_xor_sync(0xFFFFFFFFu, tmax, 1));
        tmax = fmaxf(tmax, __shfl_xor_sync(0xFFFFFFFFu, tmax, 2));
        const float m_new = fmaxf(m_run, tmax);              // finite: every tile has a valid key
        const float alpha = exp2f(m_run - m_new);
        m_run = m_new;
        float psum = 0.f;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                p[nt][e] = exp2f(p[nt][e] - m_new);
                psum += p[nt][e];
            }
        l_run = l_run * alpha + psum;
#pragma unroll
        for (int i = 0; i < NT_O; ++i) { o_acc[i][0] *= alpha; o_acc[i][1] *= alpha; }

        // ---- O += P V' ----------------------------------------------------------------------
        const uint32_t pa0 = pack_bf16(p[0][0], p[0][1]);     // keys 0..7 of the tile
        const uint32_t pa2 = pack_bf16(p[1][0], p[1][1]);     // keys 8..15
        const uint32_t vbase = sbase + TILE_BYTES;
        const int vkey = (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int np = 0; np < NT_O / 2; ++np) {
            const int chunk = np * 2 + (lane >> 4);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4_trans(b0, b1, b2, b3, vbase + vkey * ROW_BYTES + ((chunk ^ (vkey & 7)) << 4));
            mma_bf16_16816(o_acc[2 * np], pa0, 0u, pa2, 0u, b0, b1);
            mma_bf16_16816(o_acc[2 * np + 1], pa0, 0u, pa2, 0u, b2, b3);
        }
        __syncwarp();                                         // stage is refilled next iteration
    }
    cp_async_wait<0>();

    // ---- normalise, G1, store ---------------------------------------------------------------
    l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 1);
    l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 2);
    if (real_row) {
        const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
        const __nv_bfloat16* g1p = a.g1 + q_off;
        __nv_bfloat16* op = a.out + q_off;
#pragma unroll
        for (int i = 0; i < NT_O; ++i) {
            const int d = i * 8 + qcol;
            const float2 gl = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(g1p + d));
            const float o0 = o_acc[i][0] * inv * fast_sigmoid(gl.x);
            const float o1 = o_acc[i][1] * inv * fast_sigmoid(gl.y);
            *reinterpret_cast<__nv_bfloat162*>(op + d) = __floats2bfloat162_rn(o0, o1);
        }
    }
}

// Eq. 9 as a streaming pre-pass: Vg = bf16(V * sigmoid(g2)), 8 elements per thread.
__global__ void __launch_bounds__(256) gsa_value_gate_kernel(const uint4* __restrict__ V,
                                                             const uint4* __restrict__ g2,
                                                             uint4* __restrict__ Vg, int64_t n_vec) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec;
         i += (int64_t)gridDim.x * blockDim.x) {
        uint4 vv = __ldg(V + i);
        const uint4 gg = __ldg(g2 + i);
        __nv_bfloat162* v2 = reinterpret_cast<__nv_bfloat162*>(&vv);
        const __nv_bfloat162* g2v = reinterpret_cast<const __nv_bfloat162*>(&gg);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 vf = __bfloat1622float2(v2[e]), gf = __bfloat1622float2(g2v[e]);
            v2[e] = __floats2bfloat162_rn(vf.x * fast_sigmoid(gf.x), vf.y * fast_sigmoid(gf.y));
        }
        Vg[i] = vv;
    }
}

template <int DH, int G, bool FUSE_G2>
cudaError_t launch_attn_t(const AttnArgs& a0, int n_kv, cudaStream_t st) {
    constexpr int STAGES = FUSE_G2 ? 2 : 3;
    constexpr int PER_WARP = STAGES * (FUSE_G2 ? 3 : 2) * kTileKeys * DH * 2;
    AttnArgs a = a0;
    a.q_per_cta = 8 / n_kv > 0 ? 8 / n_kv : 1;
    const int warps = a.q_per_cta * n_kv;
    const size_t smem = (size_t)warps * PER_WARP;
    auto kern = gsa_sparse_attn_kernel<DH, G, FUSE_G2, STAGES>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int ctas = (a.rr.rows() + a.q_per_cta - 1) / a.q_per_cta;
    kern<<<ctas, warps * 32, smem, st>>>(a);
    ++g_launches;
    return cudaGetLastError();
}

template <int DH, bool FUSE_G2>
cudaError_t launch_attn_g(const AttnArgs& a, int G, int n_kv, cudaStream_t st) {
    switch (G) {
        case 1: return launch_attn_t<DH, 1, FUSE_G2>(a, n_kv, st);
        case 2: return launch_attn_t<DH, 2, FUSE_G2>(a, n_kv, st);
        case 4: return launch_attn_t<DH, 4, FUSE_G2>(a, n_kv, st);
        case 8: return launch_attn_t<DH, 8, FUSE_G2>(a, n_kv, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_value_gate(const __nv_bfloat16* V, const __nv_bfloat16* g2, __nv_bfloat16* Vg,
                              int64_t n_elems, cudaStream_t st) {
    const int64_t n_vec = n_elems / 8;
    if (n_vec <= 0) return cudaSuccess;
    const int blocks = (int)((n_vec + 255) / 256 < 148 * 16 ? (n_vec + 255) / 256 : 148 * 16);
    gsa_value_gate_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(V),
                                                  reinterpret_cast<const uint4*>(g2),
                                                  reinterpret_cast<uint4*>(Vg), n_vec);
    ++g_launches;
    return cudaGetLastError();
}

cudaError_t launch_sparse_attn(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* Q,
                               const __nv_bfloat16* K, const __nv_bfloat16* V,
                               const __nv_bfloat16* g1, const __nv_bfloat16* g2, const int32_t* idx,
                               const int32_t* kt, IdxLayout il, __nv_bfloat16* out, cudaStream_t st) {
    if (rr.rows() <= 0) return cudaSuccess;
    AttnArgs a;
    a.Q = Q; a.K = K; a.V = V; a.g1 = g1; a.g2 = g2; a.idx = idx; a.kt = kt; a.out = out;
    a.rr = rr; a.il = il; a.Lq = p.Lq; a.Lk = p.Lk; a.n_h = p.n_h; a.n_kv = p.n_kv; a.k_max = p.k_max;
    a.q_per_cta = 1;
    const float sc = p.sm_scale > 0.f ? p.sm_scale : 1.0f / sqrtf((float)p.d_h);
    a.scale_log2 = sc * 1.4426950408889634f;
    const int G = p.n_h / p.n_kv;
    if (p.d_h == 128) return g2 ? launch_attn_g<128, true>(a, G, p.n_kv, st) : launch_attn_g<128, false>(a, G, p.n_kv, st);
    if (p.d_h == 64) return g2 ? launch_attn_g<64, true>(a, G, p.n_kv, st) : launch_attn_g<64, false>(a, G, p.n_kv, st);
    return cudaErrorInvalidValue;
}

}  // namespace gsa
