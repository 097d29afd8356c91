// Sixteen elements per thread: the streamlined step for the paper's default block size and
// plain step (2/3/4-bit states, blocks of 128, fp32 or bf16 parameters; no L2 term in the gradient, no AdaBelief, base from the p = 0.1 quantile, xi
// drawn).
//
// Same arithmetic, element for element, as solo_step_fast_kernel (solo_fast.cuh); what changes
// is the work split.  A CTA of 128 threads owns a tile of 2048 consecutive elements, a thread
// sixteen of them, a block of 128 elements eight consecutive lanes, a warp four blocks.  The
// per-thread work that does not depend on the element count (waiting for the staged inputs,
// addressing, the level tables, the exchange with the first warp, the rounds of the selection)
// is spent once per sixteen elements instead of once per eight.
//
// This kernel processes full tiles of 16-byte aligned tensors only; every other tile is left to
// a second launch of solo_step_fast_kernel with StepArgs::only_partial set.
#pragma once

#include "solo_dispatch.h"
#include "solo_fast.cuh"

namespace solo {

constexpr int EPT16 = 16;               // elements per thread
static_assert(CTA16 * EPT16 == TILE, "same tile as the other kernels");

template <int BM, int BV>
struct Fast16Shared {
    // Sorted keys of the threads, one column per thread: row j holds the (j+2)-th smallest key.
    // Twelve rounds of popping read rows 0..11 at most.
    uint32_t sort[12][CTA16];
    float tab[16][(1 << BV) + (1 << BM)]; // per block: K_v second-moment levels, then K_m first-moment levels
    // Exchange with the first warp.  One copy is enough: xin is written before the tile's first
    // barrier and read between its two barriers, xout and xflag are written between the barriers and
    // read after the second, and nobody writes either again before passing those barriers.
    uint4 xin[16];                       // per block: bits of Delta_m', Delta_v', x_p
    float4 xout[16];                     // per block: 1/Delta_m', 1/Delta_v', 1/log2(alpha'), rounding limit
    uint32_t xflag[16];
    // per 3-bit moment and warp: the packed codes of the warp's 512 elements, for 128-bit stores
    static constexpr int N3 = (BM == 3 ? 1 : 0) + (BV == 3 ? 1 : 0);
    alignas(16) uint32_t cout[N3 > 0 ? N3 : 1][N3 > 0 ? 4 : 1][N3 > 0 ? 48 : 4];   // (a token array without 3-bit codes)
    struct Stage {
        float4 p[TILE / 4];              // 2048 parameters (bf16: the first half)
        uint4 g[TILE / 8];               // 2048 bf16 gradients
        uint32_t cm[64 * BM + 4];        // packed codes of the tile: 256 * bits bytes
        uint32_t cv[64 * BV + 4];
        float sc[3][16 + 4];             // Delta_m, Delta_v, alpha of the 16 blocks, from a 16-byte boundary
    };
    alignas(16) Stage stage[2];
    alignas(8) unsigned long long mbar[2];
};

__device__ __forceinline__ void bar_sync16(int id) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(CTA16) : "memory");
}

// Byte offsets (4 * code) of sixteen 2-bit codes in one word; see CodeOffsets.
struct CodeOffsets16x2 {
    uint32_t even, odd;
    __device__ __forceinline__ explicit CodeOffsets16x2(uint32_t c) : even(c & 0x33333333u), odd(c & 0xCCCCCCCCu) {}
    __device__ __forceinline__ uint32_t operator()(int i) const {
        const uint32_t w = (i & 1) ? odd : even;
        uint32_t top;
        asm("mul.lo.u32 %0, %1, %2;" : "=r"(top) : "r"(w), "r"(1u << (30 - 2 * i)));
        return top >> 28;
    }
};

// The thread's sixteen BITS-bit codes as two words of eight codes each, from the tile's staged
// code words (thread t owns bytes [2 * BITS * t, 2 * BITS * (t + 1)) of them).
template <int BITS>
__device__ __forceinline__ void load_codes16(const uint32_t* st, int tid, uint32_t (&h)[2]) {
    if constexpr (BITS == 2) {
        const uint32_t c = st[tid];
        h[0] = c & 0xFFFFu; h[1] = c >> 16;
    } else if constexpr (BITS == 4) {
        const uint2 c = reinterpret_cast<const uint2*>(st)[tid];
        h[0] = c.x; h[1] = c.y;
    } else {
        static_assert(BITS == 3, "2, 3 or 4 bits");
        const int cw = (6 * tid) >> 2, cs = ((6 * tid) & 3) * 8;  // 48 bits from byte 6 * tid; cs is 0 or 16
        const uint32_t w0 = st[cw], w1 = st[cw + 1];
        const uint32_t c32 = __funnelshift_r(w0, w1, cs);         // bits 0..31
        const uint32_t c16 = (w1 >> cs) & 0xFFFFu;                // bits 32..47
        h[0] = c32 & 0xFFFFFFu; h[1] = (c32 >> 24) | (c16 << 8);
    }
}
// The reverse, to the tile's codes in global memory (`tile_codes`: their first byte).  3-bit codes
// (48 bits per thread) go through `stage` (48 words of the warp) so that twelve lanes store the
// warp's 192 bytes as 128-bit words.
template <int BITS>
__device__ __forceinline__ void store_codes16(uint8_t* tile_codes, uint32_t* stage, int tid, const uint32_t (&h)[2]) {
    if constexpr (BITS == 2) {
        __stcs(reinterpret_cast<uint32_t*>(tile_codes) + tid, h[0] | (h[1] << 16));
    } else if constexpr (BITS == 4) {
        __stcs(reinterpret_cast<uint2*>(tile_codes) + tid, make_uint2(h[0], h[1]));
    } else {
        const int lane = tid & 31, warp = tid >> 5;
        unsigned short* const half = reinterpret_cast<unsigned short*>(stage) + 3 * lane;
        half[0] = (unsigned short)h[0];
        half[1] = (unsigned short)((h[0] >> 16) | (h[1] << 8));
        half[2] = (unsigned short)(h[1] >> 8);
        __syncwarp();
        if (lane < 12)
            __stcs(reinterpret_cast<uint4*>(tile_codes + warp * 192) + lane, reinterpret_cast<const uint4*>(stage)[lane]);
        __syncwarp();
    }
}

// Sorts sixteen keys so that key[0..12] are the thirteen smallest in ascending order (Batcher's
// odd-even merge sort without the one exchange that only orders key[13], key[14]).
__device__ __forceinline__ void sort16_low13(uint32_t (&k)[EPT16]) {
#define SOLO_CS(a, b) cswap(k[a], k[b])
    SOLO_CS(0, 1); SOLO_CS(2, 3); SOLO_CS(0, 2); SOLO_CS(1, 3); SOLO_CS(1, 2);
    SOLO_CS(4, 5); SOLO_CS(6, 7); SOLO_CS(4, 6); SOLO_CS(5, 7); SOLO_CS(5, 6);
    SOLO_CS(0, 4); SOLO_CS(2, 6); SOLO_CS(2, 4); SOLO_CS(1, 5); SOLO_CS(3, 7); SOLO_CS(3, 5);
    SOLO_CS(1, 2); SOLO_CS(3, 4); SOLO_CS(5, 6);
    SOLO_CS(8, 9); SOLO_CS(10, 11); SOLO_CS(8, 10); SOLO_CS(9, 11); SOLO_CS(9, 10);
    SOLO_CS(12, 13); SOLO_CS(14, 15); SOLO_CS(12, 14); SOLO_CS(13, 15); SOLO_CS(13, 14);
    SOLO_CS(8, 12); SOLO_CS(10, 14); SOLO_CS(10, 12); SOLO_CS(9, 13); SOLO_CS(11, 15); SOLO_CS(11, 13);
    SOLO_CS(9, 10); SOLO_CS(11, 12); SOLO_CS(13, 14);
    SOLO_CS(0, 8); SOLO_CS(4, 12); SOLO_CS(4, 8); SOLO_CS(2, 10); SOLO_CS(6, 14); SOLO_CS(6, 10);
    SOLO_CS(2, 4); SOLO_CS(6, 8); SOLO_CS(10, 12);
    SOLO_CS(1, 9); SOLO_CS(5, 13); SOLO_CS(5, 9); SOLO_CS(3, 11); SOLO_CS(7, 15); SOLO_CS(7, 11);
    SOLO_CS(3, 5); SOLO_CS(7, 9); SOLO_CS(11, 13);
    SOLO_CS(1, 2); SOLO_CS(3, 4); SOLO_CS(5, 6); SOLO_CS(7, 8); SOLO_CS(9, 10); SOLO_CS(11, 12);
#undef SOLO_CS
}

// Minimum / maximum over the calling lane's group of eight lanes.  Three shuffle-and-compare steps
// serve the warp's four groups at once; measured faster here than the full-mask reductions over a
// transformed value that solo_fast.cuh uses for its groups of sixteen (four REDUX plus selects for
// four groups): 294 vs 284 Gparams/s on the 7B set.
__device__ __forceinline__ uint32_t group8_min(uint32_t x) {
#pragma unroll
    for (int d = 1; d < 8; d <<= 1) x = min(x, __shfl_xor_sync(0xffffffffu, x, d));
    return x;
}
__device__ __forceinline__ uint32_t group8_max(uint32_t x) {
#pragma unroll
    for (int d = 1; d < 8; d <<= 1) x = max(x, __shfl_xor_sync(0xffffffffu, x, d));
    return x;
}

// One selection round over groups of eight lanes, as pop_round in solo_fast.cuh (columns of
// CTA16 words; at most twelve rounds, so no clamp; keys as they are, no transformed domain).
template <bool LAST>
__device__ __forceinline__ uint32_t pop_round16(uint32_t& head, int& off, const uint32_t* col, uint32_t le,
                                                uint32_t self) {
    const uint32_t tgt = group8_min(head);
    if constexpr (LAST) return tgt;
    const uint32_t nxt = col[off];
    const uint32_t upto = __ballot_sync(0xffffffffu, head == tgt) & le;
    // if (upto == self) { head = nxt; off += CTA16; }
    asm("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, %2, %3;\n\t@p mov.u32 %0, %4;\n\t@p add.s32 %1, %1, %5;\n\t}"
        : "+r"(head), "+r"(off) : "r"(upto), "r"(self), "r"(nxt), "n"(CTA16));
    return tgt;
}

// Bulk copies of one full tile's inputs into stage `fill & 1` (one thread).  With blocks of 128
// the tile's codes start on 16-byte boundaries (16 * bits bytes per block); the per-block scalars
// are copied from the boundary at or below the first.
template <int BM, int BV, bool PBF>
__device__ __forceinline__ void issue_tile_copy16(const StepArgs& a, Fast16Shared<BM, BV>& s, uint32_t fill,
                                                  const char* pt, const char* gt, int64_t jb_tile) {
    typename Fast16Shared<BM, BV>::Stage& st = s.stage[fill & 1u];
    const uint32_t bar = smem_u32(&s.mbar[fill & 1u]);
    const uint32_t bytes_s = (16u + ((jb_tile & 3) ? 4u : 0u)) * 4u;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar),
                 "r"((uint32_t)(TILE * (PBF ? 2 : 4) + TILE * 2 + 256 * BM + 256 * BV) + 3u * bytes_s) : "memory");
    bulk_copy(st.p, pt, TILE * (PBF ? 2 : 4), bar);
    bulk_copy(st.g, gt, TILE * 2, bar);
    bulk_copy(st.cm, a.codes_m + jb_tile * (16 * BM), 256 * BM, bar);
    bulk_copy(st.cv, a.codes_v + jb_tile * (16 * BV), 256 * BV, bar);
    const int64_t j0 = jb_tile & ~(int64_t)3;
    bulk_copy(st.sc[0], a.scale_m + j0, bytes_s, bar);
    bulk_copy(st.sc[1], a.scale_v + j0, bytes_s, bar);
    bulk_copy(st.sc[2], a.alpha + j0, bytes_s, bar);
}

// One full tile.  Arguments as for fast_tile.
template <int BM, int BV, bool PBF>
__device__ __forceinline__ void fast16_tile(const StepArgs& a, Fast16Shared<BM, BV>& s, const float* s_y, const float* s_mid,
                                            char* pbase, const char* gbase, const int tin, const int64_t jb_tile,
                                            const int tensor, Ahead& ah, const bool next_full,
                                            const int next_dtin) {
    constexpr int KM = 1 << BM, KV = 1 << BV, G = 8, NG = 16;     // 8 lanes per block, 16 blocks per tile
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gl = tid & (G - 1), grp = tid >> 3;

    const int64_t tile_elem0 = (int64_t)tin * TILE;
    constexpr int PSZ = PBF ? 2 : 4;                              // bytes per parameter
    char* const pt = pbase + tile_elem0 * PSZ;
    const char* const gt = gbase + tile_elem0 * 2;

    // ---- inputs from the stage (see fast_tile for the protocol) ----
    if (tid == 0) {
        if (!ah.staged) issue_tile_copy16<BM, BV, PBF>(a, s, ah.fill, pt, gt, jb_tile);
        if (next_full)
            issue_tile_copy16<BM, BV, PBF>(a, s, ah.fill + 1u, pt + (int64_t)next_dtin * (TILE * PSZ),
                              gt + (int64_t)next_dtin * (TILE * 2), jb_tile + (int64_t)next_dtin * NG);
    }
    const uint32_t mine = ah.fill;
    ah.fill += 1u;
    ah.staged = next_full;
    if (!mbar_wait(smem_u32(&s.mbar[mine & 1u]), (mine >> 1) & 1u)) {
        atomicOr(a.status, 2);
        ah.failed = true;
    }
    const typename Fast16Shared<BM, BV>::Stage& st = s.stage[mine & 1u];
    float p[EPT16], g[EPT16];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint4 gw = st.g[2 * tid + h];
        const uint32_t gg[4] = {gw.x, gw.y, gw.z, gw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            g[8 * h + 2 * i] = __uint_as_float(gg[i] << 16);
            g[8 * h + 2 * i + 1] = __uint_as_float(gg[i] & 0xffff0000u);
        }
    }
    if constexpr (PBF) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint4 pw = reinterpret_cast<const uint4*>(st.p)[2 * tid + h];
            const uint32_t pp[4] = {pw.x, pw.y, pw.z, pw.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                p[8 * h + 2 * i] = __uint_as_float(pp[i] << 16);
                p[8 * h + 2 * i + 1] = __uint_as_float(pp[i] & 0xffff0000u);
            }
        }
    } else {
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const float4 pv = st.p[4 * tid + h];
            p[4 * h] = pv.x; p[4 * h + 1] = pv.y; p[4 * h + 2] = pv.z; p[4 * h + 3] = pv.w;
        }
    }
    uint32_t cm[2], cv[2];                                        // eight codes per word
    load_codes16<BM>(st.cm, tid, cm);
    load_codes16<BV>(st.cv, tid, cv);
    const int so = (int)(jb_tile & 3) + grp;
    const float dm = st.sc[0][so], dv = st.sc[1][so], al = st.sc[2][so];

    // ---- per-block level tables (Eq. 2), built by the block's eight lanes ----
    float* const tab = s.tab[grp];
    {
        float a2[BV];
        a2[0] = al;
#pragma unroll
        for (int i = 1; i < BV; ++i) a2[i] = a2[i - 1] * a2[i - 1];
#pragma unroll
        for (int r0 = 0; r0 < KV; r0 += G) tab[r0 + gl] = pow_sm<BV>(a2, (uint32_t)(r0 + gl)) * dv;
#pragma unroll
        for (int r0 = 0; r0 < KM; r0 += G)
            if (r0 + gl < KM) tab[KV + r0 + gl] = s_y[r0 + gl] * dm;
    }
    __syncwarp();

    // ---- Eq. 2, Eq. 3 ----
    float mh[EPT16], vh[EPT16];
    uint32_t mx_v = 0;
    float mx_m_f = 0.0f;
    const char* const tab_v = reinterpret_cast<const char*>(tab);
    const char* const tab_m = reinterpret_cast<const char*>(tab + KV);
    const CodeOffsets16x2 om16(cm[0] | (cm[1] << 16));            // used for 2-bit codes only
    const CodeOffsets<BM> om4a(cm[0], 0u), om4b(cm[1], 0u);
    const CodeOffsets<BV> ov4a(cv[0], 0u), ov4b(cv[1], 0u);
#pragma unroll
    for (int i = 0; i < EPT16; ++i) {
        const float mt = *reinterpret_cast<const float*>(tab_m + (BM == 2 ? om16(i) : i < 8 ? om4a(i) : om4b(i - 8)));
        const float vt = *reinterpret_cast<const float*>(tab_v + (i < 8 ? ov4a(i) : ov4b(i - 8)));
        const float gi = g[i];
        mh[i] = __fmaf_rn(a.beta1, mt, a.omb1 * gi);
        vh[i] = __fmaf_rn(a.beta2, vt, a.omb2 * (gi * gi));
        mx_m_f = fmaxf(mx_m_f, fabsf(mh[i]));
        mx_v = max(mx_v, __float_as_uint(vh[i]));
    }
    uint32_t mx_m = __float_as_uint(mx_m_f);

    // Adam(W) update of element i; fp32 parameters are stored after every fourth.  bf16 parameters:
    // IEEE square root and division (see solo_fast.cuh), stored after every eighth, rounded to
    // nearest even or with the element's Philox draw (purpose 2, one block per eight elements)
    const uint64_t ctr = ((uint64_t)(uint32_t)tin * (TILE / 8)) + 2u * (uint32_t)tid;   // element index / 8
    auto update = [&](int i) {
        if constexpr (PBF) {
            const float den = __fmaf_rn(__fsqrt_rn(vh[i]), a.inv_sqrt_bc2, a.eps);
            p[i] = __fmaf_rn(-a.step_size, __fdiv_rn(mh[i], den), p[i] * a.decay);
            if ((i & 7) == 7) {
                const int b = i - 7;
                uint32_t pp[4];
                if (a.param_sr) {
                    uint32_t wp[4];
                    const uint64_t c = ctr + (uint64_t)(i >> 3);
                    philox_rk((uint32_t)c, (uint32_t)(c >> 32), a.step32, (uint32_t)tensor * 4u + 2u, a.rk, wp);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        pp[j] = bf16_sr(p[b + 2 * j], wp[j] & 0xFFFFu) | (bf16_sr(p[b + 2 * j + 1], wp[j] >> 16) << 16);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const __nv_bfloat162 h2 = __floats2bfloat162_rn(p[b + 2 * j], p[b + 2 * j + 1]);
                        pp[j] = *reinterpret_cast<const uint32_t*>(&h2);
                    }
                }
                __stcs(reinterpret_cast<uint4*>(pt) + 2 * tid + (i >> 3), make_uint4(pp[0], pp[1], pp[2], pp[3]));
            }
            return;
        }
        const float den = __fmaf_rn(sqrt_approx(vh[i]), a.inv_sqrt_bc2, a.eps);
        const float rc = rcp_approx(den);
        const float q0 = mh[i] * rc;
        const float q1 = __fmaf_rn(__fmaf_rn(-den, q0, mh[i]), rc, q0);
        p[i] = __fmaf_rn(-a.step_size, q1, p[i] * a.decay);
        if ((i & 3) == 3)
            __stcs(reinterpret_cast<float4*>(pt) + 4 * tid + (i >> 2), make_float4(p[i - 3], p[i - 2], p[i - 1], p[i]));
    };
    auto update2 = [&](int r) { update(2 * r); update(2 * r + 1); };

    // ---- block scales and the p-quantile (k = 13 of 128) ----
    mx_m = group8_max(mx_m);
    mx_v = group8_max(mx_v);
    uint32_t x_p;
    {
        uint32_t key[EPT16];
#pragma unroll
        for (int i = 0; i < EPT16; ++i) key[i] = __float_as_uint(vh[i]);
        sort16_low13(key);
        uint32_t* const col = &s.sort[0][tid];
#pragma unroll
        for (int j = 1; j <= 12; ++j) col[(j - 1) * CTA16] = key[j];
        // twelve rounds pop the twelve smallest keys of the block, the thirteenth minimum is x_p;
        // the parameter updates are issued between the rounds
        const uint32_t self = 1u << lane;
        const uint32_t le = (self | (self - 1u)) & (0xFFu << (lane & ~(G - 1)));
        uint32_t head = key[0];
        int off = 0;
#pragma unroll
        for (int r = 0; r < 12; ++r) {
            pop_round16<false>(head, off, col, le, self);
            if (r < 8) update2(r);
        }
        x_p = pop_round16<true>(head, off, col, le, self);
    }

    // ---- per-block scalars by the first warp; the others draw xi meanwhile ----
    if (gl == 0) s.xin[grp] = make_uint4(mx_m, mx_v, x_p, 0u);
    bar_sync16(1);
    uint32_t w[8];
    auto draw = [&]() {
        uint32_t wa[4], wb[4];
        philox_rk((uint32_t)ctr, (uint32_t)(ctr >> 32), a.step32, (uint32_t)tensor * 4u, a.rk, wa);
        philox_rk((uint32_t)(ctr + 1), (uint32_t)((ctr + 1) >> 32), a.step32, (uint32_t)tensor * 4u, a.rk, wb);
#pragma unroll
        for (int i = 0; i < 4; ++i) { w[i] = wa[i]; w[4 + i] = wb[i]; }
    };
    if (warp != 0) {
        draw();
    } else if (tid < NG) {
        const uint4 in = s.xin[tid];
        const float dm_new = __uint_as_float(in.x), dv_new = __uint_as_float(in.y);
        const bool zero_m = dm_new < TINY, zero_v = dv_new < TINY;
        const float inv_dm = 1.0f / dm_new;
        const float inv_dv = 1.0f / dv_new;
        const float rho = fminf(fmaxf(__uint_as_float(in.z) * inv_dv, RHO_MIN), RHO_MAX);
        const float lam = log2_sp(rho) * (1.0f / (float)(KV - 1));
        const float al_new = exp2_sp(lam);
        const float inv_lambda = 1.0f / log2_sp(al_new);
        const float guard = __fmaf_rn(fabsf(inv_lambda), LG2_ABS, LG2_REL * (float)(KV + 1));
        s.xout[tid] = make_float4(inv_dm, inv_dv, inv_lambda, 0.5f - guard);
        s.xflag[tid] = (zero_m ? 1u : 0u) | (zero_v ? 2u : 0u);
        const int64_t j = jb_tile + tid;
        a.scale_m[j] = zero_m ? 0.0f : dm_new;
        a.scale_v[j] = zero_v ? 0.0f : dv_new;
        a.alpha[j] = zero_v ? 0.5f : al_new;
    }
    bar_sync16(2);
    if (warp == 0) draw();
    float dr[EPT16];
#pragma unroll
    for (int i = 0; i < 8; ++i) halves_to_float(w[i], dr[2 * i], dr[2 * i + 1]);
    const float4 sc = s.xout[grp];
    const uint32_t zf = s.xflag[grp];

    // ---- first moment: nearest level (Eq. 1), see fast_tile ----
    uint32_t om[2] = {0u, 0u};                                    // eight codes per word
    {
        const float inv = sc.x;
        if constexpr (BM == 2) {
            constexpr float BIG = 0x1p100f;
            const float n0 = -s_mid[0] * BIG, n1 = -s_mid[1] * BIG, n2 = -s_mid[2] * BIG;
            float omf[2] = {0.0f, 0.0f};
#pragma unroll
            for (int i = EPT16 - 1; i >= 0; --i) {
                const float r = mh[i] * inv;
                float& acc = omf[i >> 3];
                acc = __fmaf_rn(acc, 4.0f, __saturatef(__fmaf_rn(r, BIG, n0)));
                acc += __saturatef(__fmaf_rn(r, BIG, n1));
                acc += __saturatef(__fmaf_rn(r, BIG, n2));
            }
            om[0] = (uint32_t)omf[0];
            om[1] = (uint32_t)omf[1];
        } else {
#pragma unroll
            for (int i = EPT16 - 1; i >= 0; --i) {
                const float r = mh[i] * inv;
                uint32_t q = 0;
#pragma unroll
                for (int st = KM / 2; st >= 1; st >>= 1)
                    if (r > s_mid[q + st - 1]) q += st;
                om[i >> 3] = (om[i >> 3] << BM) + q;
            }
        }
    }

    // ---- second moment: Eq. 6, see fast_tile ----
    uint32_t ov[2];
    {
        const float inv = sc.y, il = sc.z, lim = sc.w;
        constexpr float KM1 = (float)(KV - 1);
        constexpr float MAGIC = 12582912.0f;
        constexpr uint32_t MAGIC_BITS = 0x4B400000u;
        const float ils = il * (1.0f / KM1);
        const float xs1 = (float)(0x1p-16 / (KV - 1));
        const float xs0 = (float)((-0.5 + 0x1p-17) / (KV - 1));
        float worst = 0.0f;
        uint32_t acc[2] = {0u, 0u};
#pragma unroll
        for (int i = EPT16 - 1; i >= 0; --i) {
            const float r = vh[i] * inv;
            const float ts = __saturatef(__fmaf_rn(lg2_approx(r), ils, __fmaf_rn(dr[i], xs1, xs0)));
            const float u = __fmaf_rn(ts, KM1, MAGIC);
            worst = fmaxf(worst, fabsf(__fmaf_rn(ts, KM1, MAGIC - u)));
            acc[i >> 3] = acc[i >> 3] * (1u << BV) + __float_as_uint(u);
        }
        uint32_t magic_sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) magic_sum = (magic_sum << BV) + MAGIC_BITS;
        ov[0] = acc[0] - magic_sum;
        ov[1] = acc[1] - magic_sum;
        if (__any_sync(0xffffffffu, worst > lim)) {
            // too close to a rounding boundary for the approximate logarithm somewhere in the warp:
            // the exact sequence for all sixteen
            const float x1 = 0x1p-16f, x0 = -0.5f + 0x1p-17f;
            ov[0] = 0;
            ov[1] = 0;
#pragma unroll
            for (int i = EPT16 - 1; i >= 0; --i) {
                const float r = vh[i] * inv;
                uint32_t q = KV - 1;
                if (!(r < TINY)) {
                    float t = __fmaf_rn(log2_sp(r), il, __fmaf_rn(dr[i], x1, x0));
                    t = fminf(fmaxf(t, 0.0f), KM1);
                    q = (uint32_t)__float2int_rn(t);
                }
                ov[i >> 3] = (ov[i >> 3] << BV) + q;
            }
        }
    }
    if (zf & 1u) { om[0] = 0; om[1] = 0; }
    if (zf & 2u) { ov[0] = 0; ov[1] = 0; }

    // ---- store the codes ----
    store_codes16<BM>(a.codes_m + jb_tile * (16 * BM), s.cout[0][BM == 3 ? warp : 0], tid, om);
    store_codes16<BV>(a.codes_v + jb_tile * (16 * BV), s.cout[(BM == 3 && BV == 3) ? 1 : 0][BV == 3 ? warp : 0], tid, ov);
}

template <int BM, int BV, bool PBF>
__global__ void __launch_bounds__(CTA16, PBF ? 5 : 6) solo_step_fast16_kernel(const StepArgs a) {
    constexpr int KM = 1 << BM;
    extern __shared__ __align__(16) unsigned char fast16_smem[];
    Fast16Shared<BM, BV>& s = *reinterpret_cast<Fast16Shared<BM, BV>*>(fast16_smem);
    __shared__ float s_y[KM];
    __shared__ float s_mid[KM];
    const int tid = threadIdx.x;
    if (tid < KM) {
        s_y[tid] = a.tables[tid];
        if (tid < KM - 1) s_mid[tid] = a.tables[KM + tid];
    }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s.mbar[0])) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s.mbar[1])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // the tile walk of solo_step_fast_kernel (a contiguous share of the tiles per CTA); tiles that are
    // not full are skipped here
    const int launch_tiles = (int)(a.total_tiles - a.tile_first);
    const int share = (launch_tiles + (int)gridDim.x - 1) / (int)gridDim.x;
    const int tile_begin = (int)min(a.tile_first + (int64_t)blockIdx.x * share, a.total_tiles);
    const int tile_end = (int)min((int64_t)tile_begin + share, a.total_tiles);
    int tensor = (a.num_tensors > 1 && tile_begin < tile_end ? find_tensor(a.tile_start, a.num_tensors, tile_begin) : 0) - 1;
    int t_lo = 0, t_hi = 0, full_tiles = 0;
    int64_t jb0 = 0;
    char* pbase = nullptr;
    const char* gbase = nullptr;
    bool skip = false;
    Ahead ah;
    for (int tile = tile_begin; tile < tile_end; ++tile) {
        if (tile >= t_hi) {
            do {
                ++tensor;
                t_hi = (int)__ldg(a.tile_start + tensor + 1);
            } while (tile >= t_hi);
            t_lo = (int)__ldg(a.tile_start + tensor);
            const int64_t n = __ldg(a.numel + tensor);
            jb0 = __ldg(a.block_start + tensor);
            pbase = (char*)(a.param_list ? a.param_list[tensor] : a.param_single);
            gbase = (const char*)(a.grad_list ? a.grad_list[tensor] : a.grad_single);
            const bool aligned = ((((uintptr_t)pbase) | ((uintptr_t)gbase)) & 15u) == 0;
            full_tiles = aligned ? (int)(n / TILE) : 0;
            skip = a.numel_check != nullptr && __ldg(a.numel_check + tensor) != n;   // reported by the other launch
        }
        const int tin = tile - t_lo;
        if (skip || tin >= full_tiles) continue;
        fast16_tile<BM, BV, PBF>(a, s, s_y, s_mid, pbase, gbase, tin, jb0 + (int64_t)tin * 16, tensor, ah,
                    tin + 1 < full_tiles && tile + 1 < tile_end, 1);
    }
    if (tid == 0 && ah.failed && ah.fill > 0) {
        const uint32_t last = ah.fill - 1u;
        mbar_wait(smem_u32(&s.mbar[last & 1u]), (last >> 1) & 1u);
    }
}

}  // namespace solo
