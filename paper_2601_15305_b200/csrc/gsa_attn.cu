// Sparse gated attention (Eq. 9, 11, 12, 10).
//
// Work item = (query token, KV head, segment of the token's index set S_t); one warp per item,
// 16 warps per CTA, items dealt to warps round-robin so that the warps of a CTA work on the same
// two tokens.  A warp walks its segment 16 selected keys at a time:
//
//   K   the 16 keys' d_h-wide slices are read with 16-byte loads straight into the registers that
//       the tensor-core MMA takes as its A operand (keys are M).  The contraction index of Q.K is
//       d, and a sum does not care about the order of its terms, so each thread simply uses the 8
//       consecutive d it loaded as "its" k-indices and reads Q with the same permutation: no
//       shared memory, no shuffles.                          S^T[key, head] = K[key,:] . Q[head,:]
//   softmax  online, per head = per column of S^T: max/sum across the 8 lanes that hold a column.
//   P^T -> B operand: the bf16 pairs of S^T's fragment are an 8x8 matrix; one movmatrix
//       transposes it into the B-fragment layout.
//   V'  the 16 keys' slices arrive by 16-byte async copies in a private two-stage buffer in
//       shared memory and are read transposed (ldmatrix.trans) as the A operand of
//                                                          O^T[d, head] += V'^T[d, key] P^T[key, head]
//       With heads on the N side one MMA covers all G <= 8 query heads of the KV group, so the
//       whole tile costs d_h/16 + d_h/16 MMAs of m16n8k16.
//   The next tile's K loads, V' copies and indices are in flight while the current tile is
//   computed.  16 warps x (4 KB in registers + 4 KB in shared memory) per SM keep the L2 busy.
//
// The gather dominates: every selected (token, key) pair moves one K row and one V' row of all KV
// heads (4 KB at the 1.7B shape).  Random 2 KB rows come at ~8 TB/s out of HBM but at 11-13 TB/s
// out of the 126 MB L2, so for long contexts the key axis is cut into ranges whose K and V' rows
// fit in L2 and the kernel is launched once per range, over every query's sub-list in that range
// (index sets are ascending, so a sub-list is contiguous).  The online-softmax state (m, l, O) of a
// (token, head) is carried from range to range in fp32 in the workspace.  For decode-sized calls
// (few tokens) the same state slots hold the partial results of segments that run in parallel.
// A last small kernel merges the slots, normalises, applies G1 and rounds to bf16 once.
//
// G2 is either applied by a streaming pre-pass (V' = bf16(V * sigmoid(g2)), prefill) or on the gathered
// rows (decode, where gating the whole cache would cost more than the attention): the V and the g2 slices
// of a tile then arrive in two shared-memory tiles, both are read transposed into the same A-fragment
// layout, and the gate is applied to the fragments in registers right before the MMA.
#include "gsa_common.cuh"

namespace gsa {

namespace {

constexpr int kTileKeys = 16;
constexpr int kWarpsPrefill = 16;          // warps per CTA, V' pre-gated
constexpr int kWarpsFused = 16;            // warps per CTA when V and g2 are gathered raw and gated in the fragments
constexpr float kRefSlack = 8.0f;          // a score may exceed the softmax reference by 2^8 before the reference moves
constexpr int kVStages = 2;                // shared-memory stages of a warp's V' tiles (one being read, the others in flight;
                                           // measured at L = 128K: 2 stages 90.2 ms, 3 stages 94.7 ms)
constexpr int kRangeKeysDefault = 16384;   // keys per L2 range: K + V' rows of 16K tokens = 64 MB at the 1.7B shape
constexpr int kMaxRanges = 48;
constexpr int kPartKeys = 128;             // decode: fewest keys worth a parallel segment
constexpr int kMaxParts = 16;              // most segments (and state slots) per index set

struct AttnArgs {
    const __nv_bfloat16* Q;
    const __nv_bfloat16* K;
    const __nv_bfloat16* V;
    const __nv_bfloat16* g2;
    const int32_t* idx;
    const int32_t* kt;
    const int32_t* cuts;      // range mode: [idx rows][n_cuts] positions in the index row where each range starts
    float* state;             // [slots][idx rows][n_kv][G*(d_h+2)] fp32
    RowRange rr;
    IdxLayout il;
    int64_t idx_rows;         // rows of the idx / kt / state tables
    int32_t Lq, Lk, n_h, n_kv, k_max;
    int32_t mode;             // 0: one key range per launch (range index `range`), 1: parallel parts
    int32_t max_parts;        // mode 1: segments (= state slots) per index set
    int32_t range, n_cuts;
    float scale_log2;         // sm_scale * log2(e)
    float* lse;               // optional output [B, Lq, n_h]: natural log of sum_j exp(sm_scale * q.k_j) over S_t
    int32_t* dev_status;      // where an out-of-range index or budget is reported (may be null)
};

struct RowId { int32_t b, t; int64_t irow; };

__device__ __forceinline__ RowId row_of(const RowRange& rr, const IdxLayout& il, int lr) {
    RowId r;
    r.b = rr.b0 + lr / rr.R;
    r.t = rr.q_begin + lr % rr.R;
    r.irow = il.row(r.b, r.t);
    return r;
}

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// 32 bytes per thread: a warp-wide load covers whole 128-byte lines of 8 rows
__device__ __forceinline__ void ldg_stream32(const void* p, uint4& lo, uint4& hi) {
    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(lo.x), "=r"(lo.y), "=r"(lo.z), "=r"(lo.w), "=r"(hi.x), "=r"(hi.y), "=r"(hi.z), "=r"(hi.w)
                 : "l"(p));
}
__device__ __forceinline__ float ex2_fast(float x) {          // 2^x, one special-function instruction; 2^-inf = 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__host__ __device__ __forceinline__ int parts_of(int k_eff, int max_parts) {
    const int p = (k_eff + kPartKeys - 1) / kPartKeys;
    return p < 1 ? 1 : (p > max_parts ? max_parts : p);
}

template <int DH, int G, bool FUSE_G2>
__global__ void __launch_bounds__((FUSE_G2 ? kWarpsFused : kWarpsPrefill) * 32, 1)
gsa_sparse_attn_kernel(const AttnArgs a) {
    constexpr int kWarpsPerCta = FUSE_G2 ? kWarpsFused : kWarpsPrefill;
    constexpr int HEAD_BYTES = DH * 2;
    constexpr int NC = DH / 32;                         // 32-d chunks of a head row (one uint4 per thread each)
    constexpr int MT = DH / 16;                         // output m-tiles
    constexpr int VSTRIDE = HEAD_BYTES + 16;            // padded row of the staged V' tile
    constexpr int VTILE = kTileKeys * VSTRIDE;
    constexpr int VSTAGES = FUSE_G2 ? 2 : kVStages;     // fused G2: one tile of V and one of g2, each single-staged
    constexpr int CHUNKS = HEAD_BYTES / 16;             // 16-byte chunks per head row
    constexpr int KPI = 32 / CHUNKS;                    // keys one warp-wide 16-byte copy covers
    constexpr int ITS = kTileKeys / KPI;
    constexpr int STATE_F = G * (DH + 2);               // floats of one (row, KV head) state

    extern __shared__ __align__(128) unsigned char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    unsigned char* my_smem = smem + (size_t)warp * VSTAGES * VTILE;
    const uint32_t my_s32 = smem_u32(my_smem);
    const int n_kv = a.n_kv;
    const int vkey = lane / CHUNKS, vch = lane % CHUNKS;
    const bool real_head = gid < G;                     // this thread's column of Q^T is a real head
    const bool real_cols = 2 * tig < G;                 // this thread's output columns hold real heads

    const int rows = a.rr.rows();
    const int64_t n_items = (int64_t)rows * n_kv * (a.mode == 1 ? a.max_parts : 1);
    const int64_t warps_total = (int64_t)gridDim.x * kWarpsPerCta;

    for (int64_t item = (int64_t)blockIdx.x * kWarpsPerCta + warp; item < n_items; item += warps_total) {
        const int g = (int)(item % n_kv);
        int64_t rest = item / n_kv;
        int part = 0;
        if (a.mode == 1) { part = (int)(rest % a.max_parts); rest /= a.max_parts; }
        const RowId r = row_of(a.rr, a.il, (int)rest);
        const int k_eff = checked_budget(a.kt[r.irow], a.k_max, a.dev_status);
        int lo, hi, slot = 0;
        if (a.mode == 0) {
            lo = 0;
            hi = k_eff;
            if (a.n_cuts > 1) {
                const int32_t* c = a.cuts + r.irow * a.n_cuts + a.range;
                lo = c[0];
                if (a.range + 1 < a.n_cuts) hi = c[1];
            }
        } else {
            const int np = parts_of(k_eff, a.max_parts);
            if (part >= np) continue;
            const int per = ((k_eff + np - 1) / np + kTileKeys - 1) / kTileKeys * kTileKeys;
            lo = part * per;
            hi = min(k_eff, lo + per);
            slot = part;
        }
        const int count = hi - lo;
        if (count <= 0 && !(a.mode == 1)) continue;
        const int32_t* __restrict__ idx_seg = a.idx + r.irow * a.k_max + lo;
        const int ntiles = (count + kTileKeys - 1) / kTileKeys;
        float* __restrict__ st = a.state + (((int64_t)slot * a.idx_rows + r.irow) * n_kv + g) * STATE_F;

        // ---- Q^T as the B operand, in the permuted-d order the K loads use ----------------------
        uint4 qb[NC];     // piece c = bytes [(c/2)*128 + tig*32 + (c%2)*16, +16) of the head row
        {
            const int h = g * G + (real_head ? gid : 0);
            const __nv_bfloat16* qp = a.Q + (((size_t)r.b * a.Lq + r.t) * a.n_h + h) * DH + tig * 16;
#pragma unroll
            for (int c = 0; c < NC; ++c)
                qb[c] = real_head ? *reinterpret_cast<const uint4*>(qp + (c >> 1) * 64 + (c & 1) * 8)
                                  : make_uint4(0u, 0u, 0u, 0u);
        }

        // ---- state: O^T[d, head] fragments, running max and sum per head ----------------------
        float o[MT][4];
        float m_run[2], l_run[2];
        const bool carry_in = a.mode == 0 && lo > 0;
        if (carry_in && real_cols) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const int d = mt * 16 + hf * 8 + gid;
                    if (G >= 2) {
                        const float2 v = *reinterpret_cast<const float2*>(st + d * G + 2 * tig);
                        o[mt][hf * 2] = v.x; o[mt][hf * 2 + 1] = v.y;
                    } else {
                        o[mt][hf * 2] = st[d]; o[mt][hf * 2 + 1] = 0.f;
                    }
                }
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const bool ok = 2 * tig + e < G;
                m_run[e] = ok ? st[G * DH + 2 * tig + e] : -INFINITY;
                // every lane of a column accumulates its own share of l; the carried sum goes to one of them
                l_run[e] = (ok && gid == 0) ? st[G * DH + G + 2 * tig + e] : 0.f;
            }
        } else {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }
            m_run[0] = m_run[1] = -INFINITY;
            l_run[0] = l_run[1] = 0.f;
        }

        // per-item address bases: a gathered row's address is base + position * row_bytes
        const uint32_t row_bytes = (uint32_t)n_kv * HEAD_BYTES;
        const size_t head0 = ((size_t)r.b * a.Lk * n_kv + g) * HEAD_BYTES;
        const unsigned char* kbase = reinterpret_cast<const unsigned char*>(a.K) + head0 + tig * 32;
        const unsigned char* vbase = reinterpret_cast<const unsigned char*>(a.V) + head0 + vch * 16;
        const unsigned char* gbase = reinterpret_cast<const unsigned char*>(a.g2) + head0 + vch * 16;
        const uint32_t vdst = my_s32 + vkey * VSTRIDE + vch * 16;
        const int32_t pad_pos = count > 0 ? idx_seg[0] : 0;          // tail keys re-read a valid row (P = 0 there)
        auto load_pos = [&](int tile) -> int32_t {
            const int j = tile * kTileKeys + (lane & 15);
            const int32_t p = j < count ? idx_seg[j] : pad_pos;
            return checked_pos(p, a.Lk, a.dev_status);               // a corrupt index must not leave the tensor
        };
        uint4 kb[2 * NC];                                            // K tile = A operand fragments
        auto issue_k = [&](int32_t pos16) {
            const uint32_t p0 = __shfl_sync(0xFFFFFFFFu, pos16, gid), p1 = __shfl_sync(0xFFFFFFFFu, pos16, gid + 8);
            const unsigned char* k0 = kbase + (uint64_t)p0 * row_bytes;
            const unsigned char* k1 = kbase + (uint64_t)p1 * row_bytes;
#pragma unroll
            for (int c = 0; c < NC; c += 2) {
                ldg_stream32(k0 + (c >> 1) * 128, kb[c], kb[c + 1]);
                ldg_stream32(k1 + (c >> 1) * 128, kb[NC + c], kb[NC + c + 1]);
            }
        };
        // (fused G2: `stage` is ignored; the V tile sits at stage 0 and the g2 tile at stage 1)
        auto issue_v = [&](int32_t pos16, int stage) {
#pragma unroll
            for (int i = 0; i < ITS; ++i) {
                const uint32_t p = __shfl_sync(0xFFFFFFFFu, pos16, i * KPI + vkey);
                const uint64_t goff = (uint64_t)p * row_bytes;
                if (FUSE_G2) {
                    cp_async16(vdst + i * KPI * VSTRIDE, vbase + goff);
                    cp_async16(vdst + VTILE + i * KPI * VSTRIDE, gbase + goff);
                } else {
                    cp_async16(vdst + stage * VTILE + i * KPI * VSTRIDE, vbase + goff);
                }
            }
        };

        // positions of the tile whose K loads are issued next (tile + 1) and of the tile whose V' copies are
        // issued next (tile + VSTAGES - 1)
        int32_t pos_nxt = load_pos(1), pos_vahead = load_pos(VSTAGES - 1);
        {
            const int32_t pos0 = load_pos(0);
            issue_v(pos0, 0);
            cp_async_commit();
            if (!FUSE_G2) {
#pragma unroll
                for (int t = 1; t < VSTAGES - 1; ++t) {
                    if (t < ntiles) issue_v(load_pos(t), t);
                    cp_async_commit();                                   // (possibly empty: one group per tile)
                }
            }
            issue_k(pos0);
        }

        for (int tile = 0, stage = 0; tile < ntiles; ++tile, stage = (FUSE_G2 || stage == VSTAGES - 1) ? 0 : stage + 1) {
            const bool more = tile + 1 < ntiles;
            const int32_t pos_v = pos_nxt;                            // fused G2: the next tile's V / g2 copies go out after this tile's product
            if (!FUSE_G2) {
                // the stage consumed by the previous tile takes the tile after the next one
                if (tile + VSTAGES - 1 < ntiles) issue_v(pos_vahead, stage == 0 ? VSTAGES - 1 : stage - 1);
                cp_async_commit();
            }

            // ---- S^T = K Q^T : rows = 16 keys, columns = heads --------------------------------
            // (two accumulators: half the length of the dependent MMA chain)
            float s[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                mma_bf16_16816(s, kb[c].x, kb[NC + c].x, kb[c].y, kb[NC + c].y, qb[c].x, qb[c].y);
                mma_bf16_16816(s2, kb[c].z, kb[NC + c].z, kb[c].w, kb[NC + c].w, qb[c].z, qb[c].w);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) s[e] += s2[e];
            if (more) issue_k(pos_nxt);
            pos_nxt = load_pos(tile + 2);
            pos_vahead = VSTAGES == 2 ? pos_nxt : load_pos(tile + VSTAGES);

            // ---- online softmax per head (column) ------------------------------------------------
            // The reference value m_run that the exponentials are taken against need not be the running
            // maximum itself: any value that no score exceeds by more than kRefSlack (in the log2 domain) keeps
            // 2^(s - m_run) <= 2^kRefSlack, harmless in fp32 and bf16, and the normalisation at the end divides
            // it out.  So the reduction over the tile's keys (shuffles across the lanes of a column) and the
            // rescaling run only when some score jumps above the reference: on a row's first tiles.
            const int j0 = tile * kTileKeys + gid;
            const bool v0 = j0 < count, v1 = j0 + 8 < count;
            float sc[4];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                sc[e] = v0 ? s[e] * a.scale_log2 : -INFINITY;
                sc[2 + e] = v1 ? s[2 + e] * a.scale_log2 : -INFINITY;
            }
            const bool jump = fmaxf(sc[0], sc[2]) > m_run[0] + kRefSlack || fmaxf(sc[1], sc[3]) > m_run[1] + kRefSlack;
            if (__any_sync(0xFFFFFFFFu, jump)) {
                float alpha[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    float mx = fmaxf(sc[e], sc[2 + e]);
                    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 4));
                    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 8));
                    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 16));
                    const float m_new = fmaxf(m_run[e], mx);          // finite: key 0 of every tile is valid
                    alpha[e] = ex2_fast(m_run[e] - m_new);
                    m_run[e] = m_new;
                    l_run[e] *= alpha[e];
                }
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    o[mt][0] *= alpha[0]; o[mt][1] *= alpha[1]; o[mt][2] *= alpha[0]; o[mt][3] *= alpha[1];
                }
            }
            float p[4];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                p[e] = ex2_fast(sc[e] - m_run[e]);
                p[2 + e] = ex2_fast(sc[2 + e] - m_run[e]);
                l_run[e] += p[e] + p[2 + e];
            }
            // P^T[key, head] as the B operand: transpose the two 8x8 bf16 blocks of the fragment
            const uint32_t pb0 = movmatrix_trans(pack_bf16(p[0], p[1]));     // keys 0..7
            const uint32_t pb1 = movmatrix_trans(pack_bf16(p[2], p[3]));     // keys 8..15

            // ---- O^T += V'^T P^T -------------------------------------------------------------------
            if (FUSE_G2) cp_async_wait<0>(); else cp_async_wait<kVStages - 1>();   // this tile's copies have landed
            __syncwarp();
            {
                const int mi = lane >> 3;
                const uint32_t vaddr = my_s32 + (FUSE_G2 ? 0 : stage) * VTILE + ((lane & 7) + (mi >> 1) * 8) * VSTRIDE + (mi & 1) * 16;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    uint32_t a0, a1, a2, a3;
                    ldmatrix_x4_trans(a0, a1, a2, a3, vaddr + mt * 32);
                    if constexpr (FUSE_G2) {
                        // Eq. 9 on the fragments: the g2 tile read the same way has the same layout
                        uint32_t g0, g1r, g2r, g3;
                        ldmatrix_x4_trans(g0, g1r, g2r, g3, vaddr + VTILE + mt * 32);
                        auto gate = [](uint32_t v, uint32_t g) -> uint32_t {
                            const float2 vf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v));
                            const float2 gf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&g));
                            return pack_bf16(vf.x * gate_sigmoid(gf.x), vf.y * gate_sigmoid(gf.y));
                        };
                        a0 = gate(a0, g0); a1 = gate(a1, g1r); a2 = gate(a2, g2r); a3 = gate(a3, g3);
                    }
                    mma_bf16_16816(o[mt], a0, a1, a2, a3, pb0, pb1);
                }
            }
            __syncwarp();                                             // the tiles are refilled from here on
            if (FUSE_G2) {
                if (more) issue_v(pos_v, 0);
                cp_async_commit();
            }
        }
        cp_async_wait<0>();

        // ---- write the state slot ---------------------------------------------------------------
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            l_run[e] += __shfl_xor_sync(0xFFFFFFFFu, l_run[e], 4);
            l_run[e] += __shfl_xor_sync(0xFFFFFFFFu, l_run[e], 8);
            l_run[e] += __shfl_xor_sync(0xFFFFFFFFu, l_run[e], 16);
        }
        if (real_cols) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const int d = mt * 16 + hf * 8 + gid;
                    if (G >= 2) *reinterpret_cast<float2*>(st + d * G + 2 * tig) = make_float2(o[mt][hf * 2], o[mt][hf * 2 + 1]);
                    else st[d] = o[mt][hf * 2];
                }
            if (gid == 0) {
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    if (2 * tig + e < G) { st[G * DH + 2 * tig + e] = m_run[e]; st[G * DH + G + 2 * tig + e] = l_run[e]; }
            }
        }
    }
}

// cuts[row][c] = number of selected positions of the row below c * range_keys (c = 0 .. n_cuts-1)
__global__ void __launch_bounds__(256) gsa_range_cuts_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ kt,
                                                             int32_t* __restrict__ cuts, RowRange rr, IdxLayout il,
                                                             int k_max, int n_cuts, int range_keys) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)rr.rows() * n_cuts) return;
    const int c = (int)(i % n_cuts);
    const RowId r = row_of(rr, il, (int)(i / n_cuts));
    const int32_t* __restrict__ row = idx + r.irow * k_max;
    const int k_eff = clamp_budget(kt[r.irow], k_max);
    const int bound = c * range_keys;
    int lo = 0, hi = k_eff;                      // first position with row[pos] >= bound
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (row[mid] < bound) lo = mid + 1; else hi = mid;
    }
    cuts[r.irow * n_cuts + c] = lo;
}

// merge the state slots of a (row, head): out = (sum_p 2^(m_p - M) O_p) / (sum_p 2^(m_p - M) l_p) * sigmoid(g1)
// A CTA takes kFinRows consecutive query rows; thread = (KV head, d), all G heads of the group.  With a
// single slot per row (prefill) the loads of all rows are issued before any is used.
constexpr int kFinRows = 4;

template <int DH, int G>
__global__ void __launch_bounds__(1024) gsa_attn_finalize_kernel(const float* __restrict__ state, const int32_t* __restrict__ kt,
                                                                const __nv_bfloat16* __restrict__ g1, __nv_bfloat16* __restrict__ out,
                                                                RowRange rr, IdxLayout il, int64_t idx_rows, int Lq, int n_h,
                                                                int n_kv, int k_max, int mode, int max_parts,
                                                                float* __restrict__ lse) {
    constexpr int STATE_F = G * (DH + 2);
    const int rows = rr.rows();
    // range mode: kFinRows rows per CTA, all (KV head, d) pairs; parts mode (few rows, several state slots to
    // merge per row): one row and one KV head per CTA, so that a decode batch still fills the GPU
    const int rows_per_cta = mode == 0 ? kFinRows : 1;
    const int lr0 = blockIdx.x * rows_per_cta;
    const int i_begin = gridDim.y > 1 ? blockIdx.y * DH : 0, i_end = gridDim.y > 1 ? i_begin + DH : n_kv * DH;
    if (mode == 0) {
        // thread = (KV head, two consecutive d): 2 G consecutive floats of the state, bf16 pairs of g1 and out
        for (int i = threadIdx.x; i < n_kv * (DH / 2); i += blockDim.x) {
            const int d = (i % (DH / 2)) * 2;
            const int g = i / (DH / 2);
            float o[kFinRows][2 * G], l[kFinRows][G];
            __nv_bfloat162 gl[kFinRows][G];
            int keff[kFinRows];
            size_t at0[kFinRows];
#pragma unroll
            for (int q = 0; q < kFinRows; ++q) {
                const int lr = min(lr0 + q, rows - 1);
                const RowId r = row_of(rr, il, lr);
                const float* st = state + ((int64_t)r.irow * n_kv + g) * STATE_F;
                keff[q] = kt[r.irow];
                at0[q] = (((size_t)r.b * Lq + r.t) * n_h + g * G) * DH + d;
                if constexpr (G == 1) {
                    const float2 v = *reinterpret_cast<const float2*>(st + d);
                    o[q][0] = v.x; o[q][1] = v.y;
                } else {
#pragma unroll
                    for (int c = 0; c < 2 * G / 4; ++c) {
                        const float4 v = *reinterpret_cast<const float4*>(st + d * G + 4 * c);
                        o[q][4 * c] = v.x; o[q][4 * c + 1] = v.y; o[q][4 * c + 2] = v.z; o[q][4 * c + 3] = v.w;
                    }
                }
#pragma unroll
                for (int e = 0; e < G; ++e) {
                    l[q][e] = st[G * DH + G + e];
                    gl[q][e] = *reinterpret_cast<const __nv_bfloat162*>(g1 + at0[q] + (size_t)e * DH);
                }
            }
#pragma unroll
            for (int q = 0; q < kFinRows; ++q) {
                if (lr0 + q >= rows) break;
#pragma unroll
                for (int e = 0; e < G; ++e) {
                    const bool live = keff[q] > 0 && l[q][e] > 0.f;
                    const float2 gf = __bfloat1622float2(gl[q][e]);
                    const float v0 = live ? o[q][e] / l[q][e] * fast_sigmoid(gf.x) : 0.f;          // (d, head e)
                    const float v1 = live ? o[q][G + e] / l[q][e] * fast_sigmoid(gf.y) : 0.f;      // (d + 1, head e)
                    *reinterpret_cast<__nv_bfloat162*>(out + at0[q] + (size_t)e * DH) = __floats2bfloat162_rn(v0, v1);
                    if (lse && d == 0) {               // the running maximum sits in front of the sums (log2 domain)
                        const RowId r = row_of(rr, il, lr0 + q);
                        const float m = state[((int64_t)r.irow * n_kv + g) * STATE_F + G * DH + e];
                        lse[((size_t)r.b * Lq + r.t) * n_h + g * G + e] = (m + log2f(l[q][e])) * 0.6931471805599453f;
                    }
                }
            }
        }
        return;
    }
    for (int i = i_begin + threadIdx.x; i < i_end; i += blockDim.x) {
        const int d = i % DH;
        const int g = i / DH;
        {
            for (int q = 0; q < rows_per_cta && lr0 + q < rows; ++q) {
                const RowId r = row_of(rr, il, lr0 + q);
                const int k_eff = clamp_budget(kt[r.irow], k_max);
                const int np = parts_of(k_eff, max_parts);
                float acc[G], mx[G], den[G];
#pragma unroll
                for (int e = 0; e < G; ++e) { acc[e] = 0.f; den[e] = 0.f; mx[e] = -INFINITY; }
                if (k_eff > 0) {
                    for (int p = 0; p < np; ++p) {
                        const float* st = state + (((int64_t)p * idx_rows + r.irow) * n_kv + g) * STATE_F;
#pragma unroll
                        for (int e = 0; e < G; ++e) mx[e] = fmaxf(mx[e], st[G * DH + e]);
                    }
                    for (int p = 0; p < np; ++p) {
                        const float* st = state + (((int64_t)p * idx_rows + r.irow) * n_kv + g) * STATE_F;
#pragma unroll
                        for (int e = 0; e < G; ++e) {
                            const float m = st[G * DH + e];
                            const float sc = m == -INFINITY ? 0.f : exp2f(m - mx[e]);
                            acc[e] = fmaf(sc, st[d * G + e], acc[e]);
                            den[e] = fmaf(sc, st[G * DH + G + e], den[e]);
                        }
                    }
                }
#pragma unroll
                for (int e = 0; e < G; ++e) {
                    const size_t at = (((size_t)r.b * Lq + r.t) * n_h + g * G + e) * DH + d;
                    const float v = den[e] > 0.f ? acc[e] / den[e] * fast_sigmoid(__bfloat162float(g1[at])) : 0.f;
                    out[at] = __float2bfloat16_rn(v);
                    if (lse && d == 0)
                        lse[((size_t)r.b * Lq + r.t) * n_h + g * G + e] = (mx[e] + log2f(den[e])) * 0.6931471805599453f;
                }
            }
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
            v2[e] = __floats2bfloat162_rn(vf.x * gate_sigmoid(gf.x), vf.y * gate_sigmoid(gf.y));
        }
        Vg[i] = vv;
    }
}

int g_range_keys = kRangeKeysDefault;

struct AttnPlan {
    int mode;            // 0 ranges, 1 parts
    int n_ranges;        // mode 0
    int slots;
    size_t state_bytes, cuts_bytes;
};

AttnPlan plan_attn(const gsa_params_t& p) {
    AttnPlan pl;
    const int64_t idx_rows = (int64_t)p.B * p.Lq;
    const int G = p.n_h / p.n_kv;
    const size_t row_state = (size_t)p.n_kv * G * (p.d_h + 2) * 4;
    // few rows: split every index set into parallel parts; otherwise one launch per L2-sized key range
    pl.mode = idx_rows * p.n_kv < 2 * (int64_t)sm_count() * kWarpsPrefill ? 1 : 0;
    int nr = (p.Lk + g_range_keys - 1) / g_range_keys;
    if (nr > kMaxRanges) nr = kMaxRanges;
    pl.n_ranges = pl.mode == 0 ? nr : 1;
    // as many segments per index set as fill the GPU's warp slots once: one wave of longer items beat two waves of
    // shorter ones at the decode workload (attention 0.115 against 0.119 ms)
    int mp = (int)(((int64_t)sm_count() * kWarpsPrefill) / (idx_rows * p.n_kv));
    mp = mp < 1 ? 1 : (mp > kMaxParts ? kMaxParts : mp);
    pl.slots = pl.mode == 1 ? mp : 1;
    pl.state_bytes = (size_t)pl.slots * idx_rows * row_state;
    pl.cuts_bytes = pl.mode == 0 && pl.n_ranges > 1 ? (size_t)idx_rows * pl.n_ranges * 4 : 0;
    return pl;
}

template <int DH, int G, bool FUSE_G2>
cudaError_t launch_attn_t(AttnArgs a, const gsa_params_t& p, const AttnPlan& pl, const __nv_bfloat16* g1,
                          __nv_bfloat16* out, int32_t* cuts, cudaStream_t st, AttnProgress* prog) {
    constexpr int VSTAGES = FUSE_G2 ? 2 : kVStages;
    constexpr int kWarpsPerCta = FUSE_G2 ? kWarpsFused : kWarpsPrefill;
    constexpr size_t smem = (size_t)kWarpsPerCta * VSTAGES * kTileKeys * (DH * 2 + 16);
    auto kern = gsa_sparse_attn_kernel<DH, G, FUSE_G2>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int per_sm = 1;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kWarpsPerCta * 32, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    const int64_t cap = (int64_t)sm_count() * per_sm;
    const RowRange rr_all = a.rr;
    const int q_end = rr_all.q_begin + rr_all.R;
    const int off = p.Lk - p.Lq;

    if (pl.mode == 0 && pl.n_ranges > 1) {
        const int64_t n = (int64_t)rr_all.rows() * pl.n_ranges;
        gsa_range_cuts_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(a.idx, a.kt, cuts, rr_all, a.il, a.k_max,
                                                                          pl.n_ranges, g_range_keys);
        ++g_launches;
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        timeline_mark(kStageRangeCuts, st);
    }
    a.cuts = cuts;
    a.n_cuts = pl.n_ranges;
    a.mode = pl.mode;
    a.max_parts = pl.slots;
    const int fin_threads = a.n_kv * (DH / 2) < 1024 ? a.n_kv * (DH / 2) : 1024;     // range mode: two d per thread
    // normalise + G1 + bf16 for rows t_lo <= t < t_hi of every batch element, then tell the caller
    auto finalize = [&](int t_lo, int t_hi) -> cudaError_t {
        if (t_hi <= t_lo) return cudaSuccess;
        RowRange fr = rr_all;
        fr.q_begin = t_lo; fr.R = t_hi - t_lo;
        const dim3 fin_grid = pl.mode == 0 ? dim3((unsigned)((fr.rows() + kFinRows - 1) / kFinRows), 1)
                                           : dim3((unsigned)fr.rows(), (unsigned)a.n_kv);
        gsa_attn_finalize_kernel<DH, G><<<fin_grid, pl.mode == 0 ? fin_threads : DH, 0, st>>>(
            a.state, a.kt, g1, out, fr, a.il, a.idx_rows, p.Lq, p.n_h, p.n_kv, p.k_max, pl.mode, pl.slots, a.lse);
        ++g_launches;
        cudaError_t fe = cudaGetLastError();
        timeline_mark(kStageFinalize, st);
        if (fe == cudaSuccess && prog && prog->n < prog->cap && prog->n < 64) {
            fe = cudaEventRecord(prog->events[prog->n], st);
            prog->t_lo[prog->n] = t_lo; prog->t_hi[prog->n] = t_hi;
            ++prog->n;
        }
        return fe;
    };
    int finalized_to = rr_all.q_begin;                      // rows below this are final
    for (int rg = 0; rg < pl.n_ranges; ++rg) {
        AttnArgs ar = a;
        ar.range = rg;
        if (pl.mode == 0) {
            // queries that cannot see the range's first key have nothing in it
            const int t_min = rg * g_range_keys - off;
            if (t_min >= q_end) break;
            if (t_min > rr_all.q_begin) { ar.rr.q_begin = t_min; ar.rr.R = q_end - t_min; }
        }
        const int64_t items = (int64_t)ar.rr.rows() * a.n_kv * (pl.mode == 1 ? pl.slots : 1);
        const int64_t want = (items + kWarpsPerCta - 1) / kWarpsPerCta;
        const int ctas = (int)(want < cap ? want : cap);
        kern<<<ctas, kWarpsPerCta * 32, smem, st>>>(ar);
        ++g_launches;
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        timeline_mark(kStageAttn, st);
        if (pl.mode == 0 && rg + 1 < pl.n_ranges) {
            // rows whose last visible key lies in this range are complete
            const int64_t t_done = (int64_t)(rg + 1) * g_range_keys - off;
            const int t_hi = (int)(t_done < finalized_to ? finalized_to : (t_done > q_end ? q_end : t_done));
            if ((e = finalize(finalized_to, t_hi)) != cudaSuccess) return e;
            finalized_to = t_hi;
        }
    }
    return finalize(finalized_to, q_end);
}

template <int DH, bool FUSE_G2>
cudaError_t launch_attn_g(const AttnArgs& a, const gsa_params_t& p, const AttnPlan& pl, const __nv_bfloat16* g1,
                          __nv_bfloat16* out, int32_t* cuts, int G, cudaStream_t st, AttnProgress* prog) {
    switch (G) {
        case 1: return launch_attn_t<DH, 1, FUSE_G2>(a, p, pl, g1, out, cuts, st, prog);
        case 2: return launch_attn_t<DH, 2, FUSE_G2>(a, p, pl, g1, out, cuts, st, prog);
        case 4: return launch_attn_t<DH, 4, FUSE_G2>(a, p, pl, g1, out, cuts, st, prog);
        case 8: return launch_attn_t<DH, 8, FUSE_G2>(a, p, pl, g1, out, cuts, st, prog);
    }
    return cudaErrorInvalidValue;
}

}  // namespace

size_t attn_scratch_bytes(const gsa_params_t& p) {
    const AttnPlan pl = plan_attn(p);
    return (pl.state_bytes + 255) / 256 * 256 + (pl.cuts_bytes + 255) / 256 * 256;
}

void set_attn_range_keys(int keys) { g_range_keys = keys >= 1024 ? keys : kRangeKeysDefault; }
int attn_range_keys() { return g_range_keys; }

cudaError_t launch_value_gate(const __nv_bfloat16* V, const __nv_bfloat16* g2, __nv_bfloat16* Vg,
                              int64_t n_elems, cudaStream_t st) {
    const int64_t n_vec = n_elems / 8;
    if (n_vec <= 0) return cudaSuccess;
    const int blocks = (int)((n_vec + 255) / 256 < sm_count() * 16 ? (n_vec + 255) / 256 : sm_count() * 16);
    gsa_value_gate_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(V),
                                                  reinterpret_cast<const uint4*>(g2),
                                                  reinterpret_cast<uint4*>(Vg), n_vec);
    ++g_launches;
    return cudaGetLastError();
}

cudaError_t launch_sparse_attn(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* Q,
                               const __nv_bfloat16* K, const __nv_bfloat16* V,
                               const __nv_bfloat16* g1, const __nv_bfloat16* g2, const int32_t* idx,
                               const int32_t* kt, IdxLayout il, __nv_bfloat16* out, void* scratch,
                               cudaStream_t st, AttnProgress* progress, float* lse) {
    if (rr.rows() <= 0) return cudaSuccess;
    const AttnPlan pl = plan_attn(p);
    AttnArgs a;
    a.lse = lse;
    a.dev_status = t_dev_status;
    a.Q = Q; a.K = K; a.V = V; a.g2 = g2; a.idx = idx; a.kt = kt;
    a.state = reinterpret_cast<float*>(scratch);
    int32_t* cuts = reinterpret_cast<int32_t*>((char*)scratch + (pl.state_bytes + 255) / 256 * 256);
    a.cuts = cuts;
    a.rr = rr; a.il = il; a.idx_rows = (int64_t)p.B * p.Lq;
    a.Lq = p.Lq; a.Lk = p.Lk; a.n_h = p.n_h; a.n_kv = p.n_kv; a.k_max = p.k_max;
    a.mode = pl.mode; a.max_parts = pl.slots; a.range = 0; a.n_cuts = pl.n_ranges;
    const float sc = p.sm_scale > 0.f ? p.sm_scale : 1.0f / sqrtf((float)p.d_h);
    a.scale_log2 = sc * 1.4426950408889634f;
    const int G = p.n_h / p.n_kv;
    if (p.d_h == 128)
        return g2 ? launch_attn_g<128, true>(a, p, pl, g1, out, cuts, G, st, progress)
                  : launch_attn_g<128, false>(a, p, pl, g1, out, cuts, G, st, progress);
    if (p.d_h == 64)
        return g2 ? launch_attn_g<64, true>(a, p, pl, g1, out, cuts, G, st, progress)
                  : launch_attn_g<64, false>(a, p, pl, g1, out, cuts, G, st, progress);
    return cudaErrorInvalidValue;
}

}  // namespace gsa
