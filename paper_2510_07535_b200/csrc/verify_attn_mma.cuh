// Split-KV verify attention, warp-level tensor-core version (mma.sync m16n8k16, bf16 -> fp32).
//
// One CTA = 8 warps = a block of up to 128 packed rows (row r = node * G + query head in group)
// of one (sequence, KV head).  K/V tiles of 64 keys are gathered page by page with 16-byte
// cp.async copies into a 4-stage ring of XOR-swizzled shared memory; each warp owns 16 rows,
// computes S = Q K^T, applies the tree mask on tiles that reach the drafted positions, runs an
// online fp32 softmax in the exp2 domain and accumulates O += P V.  Work is cut as described in
// owl_common.cuh; a CTA whose piece covers a whole unit writes the final bf16 output itself,
// otherwise it stores a normalised fp32 partial and its LSE for the combine kernel.
//
// There are no spin waits in this kernel (cp.async groups + __syncthreads only).
#pragma once

#include "owl_common.cuh"

namespace owl {
namespace mma_path {

constexpr int kTileKeys = 64;
constexpr int kRows = 128;
constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kStages = 4;
constexpr int kTileBytes = kTileKeys * kHeadDim * 2;           // 16 KB per K or V tile
constexpr int kStageBytes = 2 * kTileBytes;
constexpr int kSchedInts = kMaxBatch + 2;                       // even, keeps what follows 8-byte aligned
constexpr int kSchedBytes = (kMaxBatch + 1) * 8 + kSchedInts * 4;
constexpr int kSmemBytes = kStages * kStageBytes + kSchedBytes + kMaxNodes * 8 + 16;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    int sz = valid ? 16 : 0;  // src-size 0 zero-fills the 16 destination bytes
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Byte offset of 16-byte chunk `ch` (0..15) of key row `key` inside a swizzled [64][128] bf16 tile.
__device__ __forceinline__ uint32_t tile_off(int key, int ch) { return (uint32_t)(key * 256 + ((ch ^ (key & 7)) << 4)); }

struct Segment {
    int b, h, mb, unit;
    int tile0, tile1;  // key tiles [tile0, tile1) of the unit
    SeqSched s;
};

// Gather one 64-key K tile and V tile of (sequence, head) into a stage.  Keys at or beyond the
// sequence's last valid position are zero-filled, so stale cache contents there never matter.
__device__ __forceinline__ void load_tile(const AttnParams& p, const Segment& g, int tile, unsigned char* stage) {
    const int tid = threadIdx.x;
    const int ch = tid & 15;
    const int keys_total = g.s.L + g.s.n;
    const uint32_t kbase = smem_u32(stage), vbase = kbase + kTileBytes;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int key = (tid >> 4) + j * 16;
        const int gk = tile * kTileKeys + key;
        bool valid = gk < keys_total;
        long long off = 0;
        if (valid) {
            int page = p.block_table[(long long)g.b * p.max_pages_per_seq + (gk >> p.page_shift)];
            if ((unsigned)page >= (unsigned)p.num_pages) {
                report(p.status, kErrBadPage);
                p.seq_bad[g.b] = p.epoch;
                valid = false;
            } else {
                off = (((long long)page * p.num_kv_heads + g.h) * p.page_size + (gk & (p.page_size - 1))) * kHeadDim + ch * 8;
            }
        }
        const uint32_t d = tile_off(key, ch);
        cp_async16(kbase + d, p.k_cache + off, valid);
        cp_async16(vbase + d, p.v_cache + off, valid);
    }
}

__device__ void process_segment(const AttnParams& p, const Segment& g, unsigned char* kv,
                                unsigned long long* s_anc, int* s_flag) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = p.group;
    const int M = g.s.n * G;

    if (!build_ancestors(p.tree_parent + g.s.node_base, g.s.n, s_anc, s_flag)) {
        if (tid == 0) { report(p.status, kErrBadTree); p.seq_bad[g.b] = p.epoch; }
        return;
    }

    // Rows of this thread: r_lo, r_lo + 8 (packed row index inside the unit).
    const int r_lo = g.mb * kRows + warp * 16 + (lane >> 2);
    const int r_hi = r_lo + 8;
    const bool warp_active = (g.mb * kRows + warp * 16) < M;

    // Q fragments (A operand) for the 8 k-steps over D, straight from global memory.
    uint32_t qf[8][4];
    {
        const int c = (lane & 3) * 2;
        const __nv_bfloat16* q_lo = nullptr;
        const __nv_bfloat16* q_hi = nullptr;
        if (r_lo < M) q_lo = p.q + ((long long)(g.s.node_base + r_lo / G) * p.num_q_heads + g.h * G + r_lo % G) * kHeadDim;
        if (r_hi < M) q_hi = p.q + ((long long)(g.s.node_base + r_hi / G) * p.num_q_heads + g.h * G + r_hi % G) * kHeadDim;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            qf[kk][0] = q_lo ? *reinterpret_cast<const uint32_t*>(q_lo + kk * 16 + c) : 0u;
            qf[kk][1] = q_hi ? *reinterpret_cast<const uint32_t*>(q_hi + kk * 16 + c) : 0u;
            qf[kk][2] = q_lo ? *reinterpret_cast<const uint32_t*>(q_lo + kk * 16 + 8 + c) : 0u;
            qf[kk][3] = q_hi ? *reinterpret_cast<const uint32_t*>(q_hi + kk * 16 + 8 + c) : 0u;
        }
    }
    const unsigned long long anc_lo = r_lo < M ? s_anc[r_lo / G] : ~0ull;
    const unsigned long long anc_hi = r_hi < M ? s_anc[r_hi / G] : ~0ull;

    float o[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
    const float scale2 = p.sm_scale * 1.4426950408889634f;

    // prologue
#pragma unroll
    for (int st = 0; st < kStages - 1; ++st) {
        if (g.tile0 + st < g.tile1) load_tile(p, g, g.tile0 + st, kv + st * kStageBytes);
        cp_async_commit();
    }

    for (int tile = g.tile0; tile < g.tile1; ++tile) {
        cp_async_wait<kStages - 2>();
        __syncthreads();
        {
            const int nxt = tile + kStages - 1;
            if (nxt < g.tile1) load_tile(p, g, nxt, kv + ((nxt - g.tile0) % kStages) * kStageBytes);
            cp_async_commit();
        }
        if (!warp_active) continue;
        unsigned char* stage = kv + ((tile - g.tile0) % kStages) * kStageBytes;
        const uint32_t kbase = smem_u32(stage), vbase = kbase + kTileBytes;

        // S = Q K^T : 16 rows x 64 keys per warp
        float s[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
            for (int k2 = 0; k2 < 4; ++k2) {
                uint32_t bf[4];
                ldmatrix_x4(bf, kbase + tile_off(nt * 8 + (lane & 7), k2 * 4 + (lane >> 3)));
                mma_bf16(s[nt], qf[k2 * 2], bf[0], bf[1]);
                mma_bf16(s[nt], qf[k2 * 2 + 1], bf[2], bf[3]);
            }
        }

        // scale into the exp2 domain; tree mask on tiles that reach the drafted positions
        const int key0 = tile * kTileKeys;
        const bool need_mask = key0 + kTileKeys > g.s.L;
        float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float x = s[nt][e] * scale2;
                if (need_mask) {
                    const int j = key0 + nt * 8 + (lane & 3) * 2 + (e & 1) - g.s.L;  // drafted index of the key
                    const unsigned long long a = (e < 2) ? anc_lo : anc_hi;
                    const bool vis = j < 0 || (j < g.s.n && ((a >> j) & 1ull));
                    if (!vis) x = -INFINITY;
                }
                s[nt][e] = x;
            }
            mx_lo = fmaxf(mx_lo, fmaxf(s[nt][0], s[nt][1]));
            mx_hi = fmaxf(mx_hi, fmaxf(s[nt][2], s[nt][3]));
        }
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
        const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
        const float mu_lo = mn_lo == -INFINITY ? 0.f : mn_lo;   // all keys so far masked: exponent base 0
        const float mu_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
        const float al_lo = fast_exp2(m_lo - mu_lo), al_hi = fast_exp2(m_hi - mu_hi);
        m_lo = mn_lo; m_hi = mn_hi;
        float sum_lo = 0.f, sum_hi = 0.f;
        uint32_t pf[4][4];  // P as A fragments for the 4 k-steps (16 keys each)
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const float p0 = fast_exp2(s[nt][0] - mu_lo), p1 = fast_exp2(s[nt][1] - mu_lo);
            const float p2 = fast_exp2(s[nt][2] - mu_hi), p3 = fast_exp2(s[nt][3] - mu_hi);
            sum_lo += p0 + p1; sum_hi += p2 + p3;
            pf[nt >> 1][(nt & 1) * 2] = pack_bf16(p0, p1);
            pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
        }
        l_lo = l_lo * al_lo + sum_lo;
        l_hi = l_hi * al_hi + sum_hi;
#pragma unroll
        for (int dn = 0; dn < 16; ++dn) { o[dn][0] *= al_lo; o[dn][1] *= al_lo; o[dn][2] *= al_hi; o[dn][3] *= al_hi; }

        // O += P V
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
            for (int dp = 0; dp < 8; ++dp) {
                uint32_t bf[4];
                ldmatrix_x4_trans(bf, vbase + tile_off(ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, dp * 2 + (lane >> 4)));
                mma_bf16(o[dp * 2], pf[ks], bf[0], bf[1]);
                mma_bf16(o[dp * 2 + 1], pf[ks], bf[2], bf[3]);
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();  // every warp is done with the ring before the next segment refills it

    if (!warp_active) return;
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    const float inv_lo = l_lo > 0.f ? 1.f / l_lo : 0.f, inv_hi = l_hi > 0.f ? 1.f / l_hi : 0.f;
    const float lse_lo = l_lo > 0.f ? (m_lo + __log2f(l_lo)) * 0.6931471805599453f : -INFINITY;
    const float lse_hi = l_hi > 0.f ? (m_hi + __log2f(l_hi)) * 0.6931471805599453f : -INFINITY;
    const int c = (lane & 3) * 2;
    const bool whole = g.tile0 == 0 && g.tile1 == g.s.tiles;
    if (whole) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = half ? r_hi : r_lo;
            if (r >= M) continue;
            const long long row = (long long)(g.s.node_base + r / G) * p.num_q_heads + g.h * G + r % G;
            const float inv = half ? inv_hi : inv_lo;
            __nv_bfloat16* dst = p.out + row * kHeadDim;
#pragma unroll
            for (int dn = 0; dn < 16; ++dn)
                *reinterpret_cast<__nv_bfloat162*>(dst + dn * 8 + c) =
                    __floats2bfloat162_rn(o[dn][half * 2] * inv, o[dn][half * 2 + 1] * inv);
            if (p.lse && (lane & 3) == 0) p.lse[row] = half ? lse_hi : lse_lo;
        }
    } else {
        const long long slot = (long long)blockIdx.x + g.unit;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = half ? r_hi : r_lo;
            if (r >= M) continue;
            const long long prow = slot * p.rows_per_slot + (r - g.mb * kRows);
            const float inv = half ? inv_hi : inv_lo;
            float* dst = p.part_o + prow * kHeadDim;
#pragma unroll
            for (int dn = 0; dn < 16; ++dn)
                *reinterpret_cast<float2*>(dst + dn * 8 + c) = make_float2(o[dn][half * 2] * inv, o[dn][half * 2 + 1] * inv);
            if ((lane & 3) == 0) p.part_lse[prow] = half ? lse_hi : lse_lo;
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1) verify_attn_mma_kernel(const AttnParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* kv = smem;
    long long* s_tile = reinterpret_cast<long long*>(smem + kStages * kStageBytes);
    int* s_unit = reinterpret_cast<int*>(s_tile + kMaxBatch + 1);
    unsigned long long* s_anc = reinterpret_cast<unsigned long long*>(s_unit + kSchedInts);
    int* s_flag = reinterpret_cast<int*>(s_anc + kMaxNodes);

    build_schedule<kTileKeys, kRows>(p, s_tile, s_unit);
    Partition part;
    part.init(s_tile[p.batch], gridDim.x);
    long long t = part.begin(blockIdx.x);
    const long long t_end = part.begin(blockIdx.x + 1);
    int b = 0;
    while (t < t_end) {
        while (s_tile[b + 1] <= t) ++b;
        Segment g;
        g.b = b;
        g.s = seq_sched<kTileKeys, kRows>(p, s_tile, s_unit, b);
        const long long local = t - g.s.tile_begin;
        const int ul = (int)(local / g.s.tiles);
        g.tile0 = (int)(local % g.s.tiles);
        const long long left = t_end - t;
        g.tile1 = (int)(g.tile0 + left < g.s.tiles ? g.tile0 + left : g.s.tiles);
        g.h = ul / g.s.row_blocks;
        g.mb = ul % g.s.row_blocks;
        g.unit = g.s.unit_begin + ul;
        process_segment(p, g, kv, s_anc, s_flag);
        t += g.tile1 - g.tile0;
    }
}

}  // namespace mma_path
}  // namespace owl
