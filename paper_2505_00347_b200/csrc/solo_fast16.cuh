// Sixteen elements per thread: the streamlined step for the plain step (2/3/4-bit states, blocks of
// 64, 128 or 256, fp32 or bf16 parameters; no L2 term in the gradient, no AdaBelief, base from the
// p = 0.1 quantile, xi drawn: MODES = 0).  Two more instantiations read other modes from the arguments:
// MODES = 1 the L2 term, AdaBelief, a fixed base, no dither; MODES = 2 also stochastic rounding of the
// first moment (Eq. 5) and the baseline second-moment codebooks (a fixed level table instead of the
// logarithmic levels: no quantile, no draws, nearest level).  (One instantiation for all of them
// measured 11 % slower on the modes of MODES = 1 than the one that leaves Eq. 5 and the tables out.)
//
// Same arithmetic, element for element, as solo_step_fast_kernel (solo_fast.cuh); what changes
// is the work split.  A CTA of 128 threads owns a tile of 2048 consecutive elements, a thread
// sixteen of them, a block of 64 / 128 / 256 elements G = 4 / 8 / 16 consecutive lanes, a warp eight,
// four or two blocks.  The per-thread work that does not depend on the element count (waiting for the
// staged inputs, addressing, the level tables, the exchange with the first warp, the rounds of the
// selection) is spent once per sixteen elements instead of once per eight.
//
// Resources are cut for seven resident CTAs per SM (28 warps): at most 72 registers per thread
// and one input stage of 13.6 KB (21.5 KB of shared memory in all).  The stage is read only
// before the tile's first CTA barrier, so the copies of the CTA's next tile are issued right after
// that barrier and land while the tile's second half (per-block scalars, random draws,
// quantization) runs.  Parameters stay in the stage until the update of their four elements needs
// them.
//
// Shared-memory banks: a thread's sixteen parameters are 64 consecutive bytes of the staged tile, so
// the eight lanes that one 128-bit shared-memory access serves hit only two groups of four banks (a
// four-way conflict; gradients, 32 bytes per thread: two-way).  Lanes 4..7 of every group of eight
// therefore take the two halves of their sixteen elements in the other order (`sw`): their accesses
// fall on the other banks, which halves the conflicts of the parameters and removes those of the
// gradients.  Everything that is tied to an element's position (its codes, its Philox draw, where
// its parameter is stored) follows the swap; nothing else depends on the order.
//
// This kernel processes full tiles of 16-byte aligned tensors only; every other tile is left to
// a second launch with StepArgs::only_partial set: of solo_step_fast_kernel, or of the general kernel
// where that one has no path (the baseline codebooks).
#pragma once

#include "solo_dispatch.h"
#include "solo_fast.cuh"

namespace solo {

constexpr int EPT16 = 16;               // elements per thread
static_assert(CTA16 * EPT16 == TILE, "same tile as the other kernels");

#ifndef SOLO_F16_MIX
#define SOLO_F16_MIX 1                  // 1: the first moment's codes are computed between the exchanges of the sort
#endif
#ifndef SOLO_F16_M3FMA
#define SOLO_F16_M3FMA 1                // 3-bit first moments: seven saturated multiply-adds instead of a 3-step table search
#endif
#ifndef SOLO_F16_M4FMA
#define SOLO_F16_M4FMA 1                // 4-bit first moments: two levels of three saturated multiply-adds
#endif
#ifndef SOLO_F16_CTAS
#define SOLO_F16_CTAS 7                 // resident CTAs per SM every instantiation is compiled for (72 registers)
#endif

// G: lanes per block (4, 8 or 16 for blocks of 64, 128 or 256 elements); NG = 128 / G blocks per tile.
template <int BM, int BV, bool PBF, int G>
struct Fast16Shared {
    static constexpr int NG = CTA16 / G;
    static constexpr int ROUNDS = G == 4 ? 6 : G == 8 ? 12 : 25;   // rank of the p = 0.1 quantile minus one: 7, 13, 26
    static constexpr int ROWS = ROUNDS < 15 ? ROUNDS : 16;         // G = 16: all fifteen further keys and a sentinel row
    // Sorted keys of the threads, one column per thread: row j holds the (j+2)-th smallest key.
    // The rounds of popping read rows 0..ROUNDS-1 at most; with 25 rounds a thread can run out of
    // keys, and row 15 holds a sentinel above every key.
    uint32_t sort[ROWS][CTA16];
    // per block: K_v second-moment levels alpha^k Delta_v and K_m first-moment levels y_k Delta_m.
    // Two arrays, so that the four blocks of a warp occupy distinct banks (up to eight levels).
    float tab_v[NG][1 << BV];
    float tab_m[NG][1 << BM];
    // Exchange with the first warp.  One copy is enough: xin is written before the tile's first
    // barrier and read between its two barriers, xout is written between the barriers and read
    // after the second, and nobody writes either again before passing those barriers.
    uint4 xin[NG];                       // per block: bits of Delta_m', Delta_v', x_p; .w != 0: the block's warp skips the tile
    float4 xout[NG];                     // per block: vanishing Delta_v' (1 or 0), 1/Delta_v', 1/log2(alpha'), rounding limit
    // per 3-bit moment and warp: the packed codes of the warp's 512 elements, for 128-bit stores
    static constexpr int N3 = (BM == 3 ? 1 : 0) + (BV == 3 ? 1 : 0);
    alignas(16) uint32_t cout[N3 > 0 ? N3 : 1][N3 > 0 ? 4 : 1][N3 > 0 ? 48 : 4];   // (a token array without 3-bit codes)
    struct Stage {
        alignas(16) unsigned char p[TILE * (PBF ? 2 : 4)];   // 2048 parameters
        alignas(16) unsigned char g[TILE * 2];                // 2048 bf16 gradients
        uint32_t cm[64 * BM + 4];        // packed codes of the tile: 256 * bits bytes, from a 16-byte boundary
        uint32_t cv[64 * BV + 4];
        float sc[3][NG + 4];             // Delta_m, Delta_v, alpha of the tile's blocks, from a 16-byte boundary
    };
    alignas(16) Stage stage;
    alignas(8) unsigned long long mbar;
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
// code words (thread t owns bytes [2 * BITS * t, 2 * BITS * (t + 1)) of them).  sw = 1: the two
// words are exchanged (h[0] then holds elements 8..15).
template <int BITS>
__device__ __forceinline__ void load_codes16(const uint32_t* st, int tid, uint32_t sw, uint32_t (&h)[2]) {
    if constexpr (BITS == 2) {
        const uint32_t c = __funnelshift_r(st[tid], st[tid], 16u * sw);
        h[0] = c & 0xFFFFu; h[1] = c >> 16;
    } else if constexpr (BITS == 4) {
        const uint2 c = reinterpret_cast<const uint2*>(st)[tid];
        h[0] = sw ? c.y : c.x; h[1] = sw ? c.x : c.y;
    } else {
        static_assert(BITS == 3, "2, 3 or 4 bits");
        const int cw = (6 * tid) >> 2, cs = ((6 * tid) & 3) * 8;  // 48 bits from byte 6 * tid; cs is 0 or 16
        const uint32_t w0 = st[cw], w1 = st[cw + 1];
        const uint32_t c32 = __funnelshift_r(w0, w1, cs);         // bits 0..31
        const uint32_t c16 = (w1 >> cs) & 0xFFFFu;                // bits 32..47
        const uint32_t lo = c32 & 0xFFFFFFu, hi = (c32 >> 24) | (c16 << 8);
        h[0] = sw ? hi : lo; h[1] = sw ? lo : hi;
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
        // the warp's 192 bytes: 128-bit words where the tile's codes start on a 16-byte boundary, else
        // (3-bit codes of 64-element blocks, 24 bytes each, from an odd block on) 64-bit words
        uint8_t* const dst = tile_codes + warp * 192;
        if ((reinterpret_cast<uintptr_t>(tile_codes) & 15u) == 0) {
            if (lane < 12) __stcs(reinterpret_cast<uint4*>(dst) + lane, reinterpret_cast<const uint4*>(stage)[lane]);
        } else {
            if (lane < 24) __stcs(reinterpret_cast<uint2*>(dst) + lane, reinterpret_cast<const uint2*>(stage)[lane]);
        }
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

// The same network as a list, for callers that issue other work between its exchanges.
__device__ constexpr unsigned char SORT16_PAIRS[62][2] = {
    {0, 1}, {2, 3}, {0, 2}, {1, 3}, {1, 2}, {4, 5}, {6, 7}, {4, 6}, {5, 7}, {5, 6},
    {0, 4}, {2, 6}, {2, 4}, {1, 5}, {3, 7}, {3, 5}, {1, 2}, {3, 4}, {5, 6},
    {8, 9}, {10, 11}, {8, 10}, {9, 11}, {9, 10}, {12, 13}, {14, 15}, {12, 14}, {13, 15}, {13, 14},
    {8, 12}, {10, 14}, {10, 12}, {9, 13}, {11, 15}, {11, 13}, {9, 10}, {11, 12}, {13, 14},
    {0, 8}, {4, 12}, {4, 8}, {2, 10}, {6, 14}, {6, 10}, {2, 4}, {6, 8}, {10, 12},
    {1, 9}, {5, 13}, {5, 9}, {3, 11}, {7, 15}, {7, 11}, {3, 5}, {7, 9}, {11, 13},
    {1, 2}, {3, 4}, {5, 6}, {7, 8}, {9, 10}, {11, 12}};

// Minimum / maximum over the calling lane's group of G lanes.  The shuffle-and-compare steps serve
// all groups of the warp at once; for groups of eight measured faster here than the full-mask reductions
// over a transformed value that solo_fast.cuh uses for its groups of sixteen (four REDUX plus selects for
// four groups): 294 vs 284 Gparams/s on the 7B set.
template <int G>
__device__ __forceinline__ uint32_t group_min16(uint32_t x) {
#pragma unroll
    for (int d = 1; d < G; d <<= 1) x = min(x, __shfl_xor_sync(0xffffffffu, x, d));
    return x;
}
template <int G>
__device__ __forceinline__ uint32_t group_max16(uint32_t x) {
#pragma unroll
    for (int d = 1; d < G; d <<= 1) x = max(x, __shfl_xor_sync(0xffffffffu, x, d));
    return x;
}

// Minimum of the group's keys as each lane holds them.  Groups of sixteen: the two groups of a warp are
// served by one full-mask minimum and one maximum, the upper group (`hi`) holding its keys complemented
// (its minimum is the complement of the warp's maximum; keys are 31-bit, so the lower group's keys stay
// below and the upper group's above 2^31); a lane holds the minimum iff its own value equals the result.
template <int G>
__device__ __forceinline__ uint32_t group_min16k(uint32_t x, bool hi) {
    if constexpr (G == 16) {
        const uint32_t lo = __reduce_min_sync(0xffffffffu, x);
        const uint32_t up = __reduce_max_sync(0xffffffffu, x);
        return hi ? up : lo;
    } else {
        return group_min16<G>(x);
    }
}

// One selection round over groups of G lanes, as pop_round in solo_fast.cuh (columns of CTA16 words;
// keys as they are, or complemented in the upper group of sixteen).  CLAMP: the offset stops at the
// sentinel row (needed when a thread can be asked for more keys than it has).
template <int G, bool LAST, bool CLAMP>
__device__ __forceinline__ uint32_t pop_round16(uint32_t& head, int& off, const uint32_t* col, uint32_t le,
                                                uint32_t self, bool hi) {
    const uint32_t tgt = group_min16k<G>(head, hi);
    if constexpr (LAST) return tgt;
    const uint32_t nxt = col[off];
    const uint32_t upto = __ballot_sync(0xffffffffu, head == tgt) & le;
    // if (upto == self) { head = nxt; off += CTA16; }
    asm("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, %2, %3;\n\t@p mov.u32 %0, %4;\n\t@p add.s32 %1, %1, %5;\n\t}"
        : "+r"(head), "+r"(off) : "r"(upto), "r"(self), "r"(nxt), "n"(CTA16));
    if constexpr (CLAMP) off = min(off, 15 * CTA16);
    return tgt;
}

// Bulk copies of one full tile's inputs into the stage (one thread; a bulk copy is a warp-wide
// instruction, so copies issued by many lanes would be serialised lane by lane).  The per-block
// scalars are copied from the 16-byte boundary at or below the first.
// `extra_tx`: bytes announced on top of what is copied (test hook: the wait for this tile then runs out).
template <int BM, int BV, bool PBF, int G>
__device__ __forceinline__ void issue_tile_copy16(const StepArgs& a, Fast16Shared<BM, BV, PBF, G>& s, const char* pt,
                                                  const char* gt, int64_t jb_tile, uint32_t extra_tx) {
    constexpr int NG = CTA16 / G;
    typename Fast16Shared<BM, BV, PBF, G>::Stage& st = s.stage;
    const uint32_t bar = smem_u32(&s.mbar);
    // byte offsets of the tile's codes (2 * G * bits bytes per block); only 3-bit codes in blocks of 64
    // (24 bytes) can start 8 bytes off a 16-byte boundary: they are copied from the boundary below, with
    // 16 bytes more (the state's arrays carry that slack), and read with an offset
    const int64_t bm0 = jb_tile * (2 * G * BM), bv0 = jb_tile * (2 * G * BV);
    const uint32_t bytes_m = 256 * BM + ((bm0 & 15) ? 16u : 0u), bytes_v = 256 * BV + ((bv0 & 15) ? 16u : 0u);
    const uint32_t bytes_s = (NG + ((jb_tile & 3) ? 4u : 0u)) * 4u;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar),
                 "r"((uint32_t)(TILE * (PBF ? 2 : 4) + TILE * 2) + bytes_m + bytes_v + 3u * bytes_s + extra_tx)
                 : "memory");
    bulk_copy(st.p, pt, TILE * (PBF ? 2 : 4), bar);
    bulk_copy(st.g, gt, TILE * 2, bar);
    bulk_copy(st.cm, a.codes_m + (bm0 & ~(int64_t)15), bytes_m, bar);
    bulk_copy(st.cv, a.codes_v + (bv0 & ~(int64_t)15), bytes_v, bar);
    const int64_t j0 = jb_tile & ~(int64_t)3;
    bulk_copy(st.sc[0], a.scale_m + j0, bytes_s, bar);
    bulk_copy(st.sc[1], a.scale_v + j0, bytes_s, bar);
    bulk_copy(st.sc[2], a.alpha + j0, bytes_s, bar);
}

// What a CTA carries from one full tile to the next.
struct Ahead16 {
    uint32_t fill = 0;        // number of the next copy to wait for (uniform over the CTA); its parity is the phase
    bool staged = false;      // that copy has already been issued (uniform)
    bool failed = false;      // this thread once waited in vain for a copy: it waits no longer and stores nothing
};

// Per-block scalars of the tile's sixteen blocks (one block per calling thread, tid = 0..15), from
// what the blocks' lanes left in xin: stores Delta_m', Delta_v', alpha' of the blocks whose warp did not
// skip the tile and leaves what Eq. 6 needs in xout.
template <int KV, class Shared>
__device__ __forceinline__ void block_scalars16(const StepArgs& a, Shared& s, const int64_t jb_tile, const int tid,
                                                const bool fixed_base, const bool vtab) {
    const uint4 in = s.xin[tid];
    const float dm_new = __uint_as_float(in.x), dv_new = __uint_as_float(in.y);
    const bool zero_m = dm_new < TINY, zero_v = dv_new < TINY;
    const float inv_dv = __frcp_rn(dv_new);
    const float rho = fminf(fmaxf(__uint_as_float(in.z) * inv_dv, RHO_MIN), RHO_MAX);
    const float lam = log2_sp(rho) * (1.0f / (float)(KV - 1));
    // (a baseline codebook has no base: the array keeps its initial 1/2)
    const float al_new = vtab ? 0.5f : fixed_base ? a.fixed_alpha : exp2_sp(lam);
    const float inv_lambda = __frcp_rn(log2_sp(al_new));
    const float guard = __fmaf_rn(fabsf(inv_lambda), LG2_ABS, LG2_REL * (float)(KV + 1));
    s.xout[tid] = make_float4(zero_v ? 1.0f : 0.0f, inv_dv, inv_lambda, 0.5f - guard);
    if (in.w == 0u) {
        const int64_t j = jb_tile + tid;
        a.scale_m[j] = zero_m ? 0.0f : dm_new;
        a.scale_v[j] = zero_v ? 0.0f : dv_new;
        a.alpha[j] = zero_v ? 0.5f : al_new;
    }
}

// One full tile.  DECAY: the parameter is multiplied by 1 - lr * wd (false: that factor is 1).
//
// Order of the work, chosen so that at most the two moments and the sort keys (48 registers) are
// live at once: (A) inputs, Eq. 2-3; (B) the parameter update, parameters read from the stage four
// at a time; (C) the first moment's scale and codes (each thread divides for itself: the scale is
// known to all eight lanes after the maximum); (D) the sort and the selection rounds, with the Philox
// rounds of the thread's two blocks of draws issued between them (they depend on nothing); (E) the
// exchange with the first warp, the second moment's codes, the stores.
template <int BM, int BV, bool PBF, int G, bool DECAY, int MODES>
__device__ __forceinline__ void fast16_tile(const StepArgs& a, Fast16Shared<BM, BV, PBF, G>& s, const float* s_y, const float* s_mid,
                                            const float4* s_mid4, const float* s_yv, const float4* s_nv,
                                            const float2* s_yg, const float4* s_br,
                                            char* pbase, const char* gbase, const int tin, const int64_t jb_tile,
                                            const int tensor, Ahead16& ah, const bool next_full, const int64_t tile_no) {
    using Shared = Fast16Shared<BM, BV, PBF, G>;
    constexpr int KM = 1 << BM, KV = 1 << BV, NG = Shared::NG;    // G lanes per block, NG blocks per tile
    constexpr int ROUNDS = Shared::ROUNDS;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gl = tid & (G - 1), grp = tid / G;
    const uint32_t sw = ((uint32_t)tid >> 2) & 1u;               // 1: this thread takes elements 8..15 first (see the top of the file)
    // PLAIN: the step of the paper as it stands (no L2 term in the gradient, no AdaBelief, base from the
    // p-quantile, xi drawn); the other instantiations read these modes from the arguments, EXT also
    // Eq. 5 and the baseline codebooks
    constexpr bool PLAIN = MODES == 0, EXT = MODES == 2;
    const bool l2 = !PLAIN && a.l2, belief = !PLAIN && a.belief;
    // baseline codebook for the second moment: levels s_yv, nearest level by the midpoints in s_nv
    const bool vtab = EXT && a.tables_v != nullptr;
    const bool fixed_base = !PLAIN && (a.fixed_alpha > 0.0f || vtab);   // no quantile to find
    const bool round_v = PLAIN || (a.round_v && !vtab);
    const bool round_m = EXT && a.round_m;                     // Eq. 5 instead of Eq. 1 for the first moment

    const int64_t tile_elem0 = (int64_t)tin * TILE;
    constexpr int PSZ = PBF ? 2 : 4;                              // bytes per parameter
    char* const pt = pbase + tile_elem0 * PSZ;
    const char* const gt = gbase + tile_elem0 * 2;

    // ---- (A) inputs from the stage ----
    // Copy number f completes phase f of the stage's mbarrier (parity f & 1).  The copy for this tile
    // was issued after the first barrier of the tile before it (ah.staged), or is issued now (the
    // CTA's first full tile, or the first after a tensor change or a tile that was not full): every
    // thread has passed both barriers of the last tile that used the stage, so nobody reads it still.
    if (!ah.staged && tid == 0)
        issue_tile_copy16<BM, BV, PBF, G>(a, s, pt, gt, jb_tile, tile_no + 1 == a.debug_stall_tile_p1 ? 16u : 0u);
    const uint32_t mine = ah.fill;
    ah.fill += 1u;
    ah.staged = next_full;
    if (!mbar_wait(smem_u32(&s.mbar), mine & 1u, ah.failed ? 1 : MBAR_POLLS)) {
        if (!ah.failed) atomicOr(a.status, 2);
        ah.failed = true;
    }
    // A warp in which any lane gave up leaves the tile alone: it stores nothing, flags its four blocks
    // for the first warp (which stores the per-block scalars), and only keeps the CTA's barriers, the
    // copy-ahead and, if it is the first warp, the other warps' scalars going.
    if (__any_sync(0xffffffffu, ah.failed)) {
        if (gl == 0) s.xin[grp] = make_uint4(0u, 0u, 0u, 1u);
        bar_sync16(1);
        if (next_full && tid == 32)
            issue_tile_copy16<BM, BV, PBF, G>(a, s, pt + TILE * PSZ, gt + TILE * 2, jb_tile + NG,
                                           tile_no + 2 == a.debug_stall_tile_p1 ? 16u : 0u);
        if (tid < NG) block_scalars16<KV>(a, s, jb_tile, tid, fixed_base, vtab);
        bar_sync16(2);
        return;
    }

    const typename Shared::Stage& st = s.stage;
    float mh[EPT16], vh[EPT16];
    uint32_t mx_v = 0;
    float mx_m_f = 0.0f;
    {
        uint32_t cm[2], cv[2];                                    // eight codes per word
        // (word offsets of codes that do not start on a 16-byte boundary: 0 or 2, see issue_tile_copy16)
        load_codes16<BM>(st.cm + ((int)((jb_tile * (2 * G * BM)) & 15) >> 2), tid, sw, cm);
        load_codes16<BV>(st.cv + ((int)((jb_tile * (2 * G * BV)) & 15) >> 2), tid, sw, cv);
        const int so = (int)(jb_tile & 3) + grp;
        const float dm = st.sc[0][so], dv = st.sc[1][so], al = st.sc[2][so];

        // per-block level tables (Eq. 2), built by the block's eight lanes
        float* const tab_vf = s.tab_v[grp];
        float* const tab_mf = s.tab_m[grp];
        {
            float a2[BV];
            a2[0] = al;
#pragma unroll
            for (int i = 1; i < BV; ++i) a2[i] = a2[i - 1] * a2[i - 1];
#pragma unroll
            for (int r0 = 0; r0 < KV; r0 += G)
                if (r0 + gl < KV) tab_vf[r0 + gl] = (vtab ? s_yv[r0 + gl] : pow_sm<BV>(a2, (uint32_t)(r0 + gl))) * dv;
#pragma unroll
            for (int r0 = 0; r0 < KM; r0 += G)
                if (r0 + gl < KM) tab_mf[r0 + gl] = s_y[r0 + gl] * dm;
        }
        __syncwarp();

        // Eq. 2, Eq. 3
        const char* const tab_v = reinterpret_cast<const char*>(tab_vf);
        const char* const tab_m = reinterpret_cast<const char*>(tab_mf);
        const CodeOffsets16x2 om16(cm[0] | (cm[1] << 16));        // used for 2-bit codes only
        const CodeOffsets<BM> om4a(cm[0], 0u), om4b(cm[1], 0u);
        const CodeOffsets<BV> ov4a(cv[0], 0u), ov4b(cv[1], 0u);
        const unsigned char* const sgb = st.g + 32 * tid;
        const uint4* const sg[2] = {reinterpret_cast<const uint4*>(sgb + 16u * sw),
                                    reinterpret_cast<const uint4*>(sgb + 16u - 16u * sw)};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint4 gw = *sg[h];
            const uint32_t gg[4] = {gw.x, gw.y, gw.z, gw.w};
            float g8[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
                g8[k] = __uint_as_float((k & 1) ? (gg[k >> 1] & 0xffff0000u) : (gg[k >> 1] << 16));
            if (l2) {                                             // Adam: the decay term joins the gradient
                float p8[8];
                if constexpr (PBF) {
                    const uint4 pw = reinterpret_cast<const uint4*>(st.p)[2 * tid + ((uint32_t)h ^ sw)];
                    const uint32_t pin[4] = {pw.x, pw.y, pw.z, pw.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        p8[2 * k] = __uint_as_float(pin[k] << 16);
                        p8[2 * k + 1] = __uint_as_float(pin[k] & 0xffff0000u);
                    }
                } else {
                    const float4* const ph = reinterpret_cast<const float4*>(st.p + 64 * tid + 32u * ((uint32_t)h ^ sw));
                    const float4 pa = ph[0], pb = ph[1];
                    p8[0] = pa.x; p8[1] = pa.y; p8[2] = pa.z; p8[3] = pa.w;
                    p8[4] = pb.x; p8[5] = pb.y; p8[6] = pb.z; p8[7] = pb.w;
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) g8[k] = __fmaf_rn(a.weight_decay, p8[k], g8[k]);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int i = 8 * h + k;
                const float gi = g8[k];
                const float mt = *reinterpret_cast<const float*>(tab_m + (BM == 2 ? om16(i) : i < 8 ? om4a(i) : om4b(i - 8)));
                const float vt = *reinterpret_cast<const float*>(tab_v + (i < 8 ? ov4a(i) : ov4b(i - 8)));
                mh[i] = __fmaf_rn(a.beta1, mt, a.omb1 * gi);
                if (belief) {                                     // AdaBelief: (g - m^)^2, plus eps
                    const float sig = gi - mh[i];
                    vh[i] = __fmaf_rn(a.beta2, vt, a.omb2 * (sig * sig)) + a.eps;
                } else {
                    vh[i] = __fmaf_rn(a.beta2, vt, a.omb2 * (gi * gi));
                }
                mx_m_f = max_abs_nan(mx_m_f, mh[i]);
                mx_v = max(mx_v, __float_as_uint(vh[i]));
            }
        }
    }

    // ---- (B) Adam(W) update, four (fp32) or eight (bf16) elements at a time ----
    // bf16 parameters: IEEE square root and division (see solo_fast.cuh), rounded to nearest even or
    // with the element's Philox draw (purpose 2, one block per eight elements)
    // position of the thread's first element in the tensor's random stream (element index / 8): even,
    // so the second group of eight never carries into the high word
    auto stream_position = [&](uint32_t& lo, uint32_t& hi, uint32_t& c3) {
        const Origin org = origin_of(a, tensor);
        const uint64_t ctr = org.ctr0 + (uint64_t)((uint32_t)tin * (TILE / 8) + 2u * (uint32_t)tid);
        lo = (uint32_t)ctr;
        hi = (uint32_t)(ctr >> 32);
        c3 = org.stream * 4u;
    };
    if constexpr (!PBF) {
        // the thread's first eight elements (in its own order) at `sp[0]`, the others at `sp[1]`
        const unsigned char* const spb = st.p + 64 * tid;
        char* const gpb = pt + 64 * tid;
        const float4* const sp[2] = {reinterpret_cast<const float4*>(spb + 32u * sw),
                                     reinterpret_cast<const float4*>(spb + 32u - 32u * sw)};
        float4* const gp[2] = {reinterpret_cast<float4*>(gpb + 32u * sw), reinterpret_cast<float4*>(gpb + 32u - 32u * sw)};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float4 pv = sp[q >> 1][q & 1];
            float p[4] = {pv.x, pv.y, pv.z, pv.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int i = 4 * q + k;
                const float den = __fmaf_rn(sqrt_approx(vh[i]), a.inv_sqrt_bc2, a.eps);
                const float rc = rcp_approx(den);
                const float q0 = mh[i] * rc;
                const float q1 = __fmaf_rn(__fmaf_rn(-den, q0, mh[i]), rc, q0);
                p[k] = __fmaf_rn(-a.step_size, q1, DECAY ? p[k] * a.decay : p[k]);
            }
            __stcs(gp[q >> 1] + (q & 1), make_float4(p[0], p[1], p[2], p[3]));
        }
    } else {
        const uint4* const sp = reinterpret_cast<const uint4*>(st.p) + 2 * tid;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t he = (uint32_t)h ^ sw;
            const uint4 pw = sp[he];
            const uint32_t pin[4] = {pw.x, pw.y, pw.z, pw.w};
            float p[8];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                p[2 * k] = __uint_as_float(pin[k] << 16);
                p[2 * k + 1] = __uint_as_float(pin[k] & 0xffff0000u);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int i = 8 * h + k;
                const float den = __fmaf_rn(__fsqrt_rn(vh[i]), a.inv_sqrt_bc2, a.eps);
                p[k] = __fmaf_rn(-a.step_size, __fdiv_rn(mh[i], den), DECAY ? p[k] * a.decay : p[k]);
            }
            uint32_t pp[4];
            if (a.param_sr) {
                uint32_t wp[4], ctr_lo, ctr_hi, c3;
                stream_position(ctr_lo, ctr_hi, c3);
                philox_rk(ctr_lo + he, ctr_hi, a.step32, c3 + 2u, a.rk, wp);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    pp[k] = bf16_sr(p[2 * k], wp[k] & 0xFFFFu) | (bf16_sr(p[2 * k + 1], wp[k] >> 16) << 16);
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const __nv_bfloat162 h2 = __floats2bfloat162_rn(p[2 * k], p[2 * k + 1]);
                    pp[k] = *reinterpret_cast<const uint32_t*>(&h2);
                }
            }
            __stcs(reinterpret_cast<uint4*>(pt) + 2 * tid + he, make_uint4(pp[0], pp[1], pp[2], pp[3]));
        }
    }

    // ---- (C) first moment: block scale, nearest level (Eq. 1), see fast_tile ----
    const uint32_t mx_m = group_max16<G>(__float_as_uint(mx_m_f));
    uint32_t om[2] = {0u, 0u};                                    // eight codes per word
    const float dm_new = __uint_as_float(mx_m);
    const float inv_m = __frcp_rn(dm_new);
    // BM == 2: code = number of midpoints below r, each comparison as the saturation of
    // (r - mid) * 2^100 on the FMA pipe (exactly 0 or 1, see fast_tile), accumulated in binary32
    constexpr float BIG = 0x1p100f;
    const float n0 = -s_mid[0] * BIG, n1 = -s_mid[1] * BIG, n2 = -s_mid[BM == 2 ? 2 : 1] * BIG;
    constexpr bool M3_FMA = BM == 3 && SOLO_F16_M3FMA;           // 3-bit: all seven comparisons that way (24 bits per word: exact)
    float n3[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    if constexpr (M3_FMA) {
#pragma unroll
        for (int k = 0; k < 4; ++k) n3[k] = -s_mid[3 + k] * BIG;
    }
    // 4-bit: the same comparisons in two levels of three: mid[3], mid[7], mid[11] give the quarter s of
    // the codebook, the three midpoints inside it come from a table row addressed by s (s_mid4, scaled
    // like n0..n2); code = 4 s + their count.  Four codes (16 bits) per binary32 accumulator.
    constexpr bool M4_FMA = BM == 4 && SOLO_F16_M4FMA;
    float nq[3] = {0.0f, 0.0f, 0.0f};
    if constexpr (M4_FMA) {
        nq[0] = -s_mid[3] * BIG; nq[1] = -s_mid[7] * BIG; nq[2] = -s_mid[11] * BIG;
    }
    float omf4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    float omf[2] = {0.0f, 0.0f};
    auto quant_m = [&](int i) {                                   // call with i = 15, 14, ..., 0
        const float r = mh[i] * inv_m;
        if constexpr (BM == 2) {
            float& acc = omf[i >> 3];
            acc = __fmaf_rn(acc, 4.0f, __saturatef(__fmaf_rn(r, BIG, n0)));
            acc += __saturatef(__fmaf_rn(r, BIG, n1));
            acc += __saturatef(__fmaf_rn(r, BIG, n2));
        } else if constexpr (M3_FMA) {
            float& acc = omf[i >> 3];
            acc = __fmaf_rn(acc, 8.0f, __saturatef(__fmaf_rn(r, BIG, n0)));
            acc += __saturatef(__fmaf_rn(r, BIG, n1));
            acc += __saturatef(__fmaf_rn(r, BIG, -s_mid[2] * BIG));
#pragma unroll
            for (int k = 0; k < 4; ++k) acc += __saturatef(__fmaf_rn(r, BIG, n3[k]));
        } else if constexpr (M4_FMA) {
            const float c0 = __saturatef(__fmaf_rn(r, BIG, nq[0]));
            const float c1 = __saturatef(__fmaf_rn(r, BIG, nq[1]));
            const float c2 = __saturatef(__fmaf_rn(r, BIG, nq[2]));
            // 2^23 + 16 s: the low bits of the pattern are the byte offset of row s
            const float t = __fmaf_rn(c2, 16.0f, __fmaf_rn(c1, 16.0f, __fmaf_rn(c0, 16.0f, 8388608.0f)));
            const float4 row = *reinterpret_cast<const float4*>(reinterpret_cast<const char*>(s_mid4) + (__float_as_uint(t) & 0x30u));
            const float sq = (c0 + c1) + c2;
            float code = __fmaf_rn(sq, 4.0f, __saturatef(__fmaf_rn(r, BIG, row.x)));
            code += __saturatef(__fmaf_rn(r, BIG, row.y));
            code += __saturatef(__fmaf_rn(r, BIG, row.z));
            omf4[i >> 2] = __fmaf_rn(omf4[i >> 2], 16.0f, code);
        } else {
            uint32_t q = 0;
#pragma unroll
            for (int st2 = KM / 2; st2 >= 1; st2 >>= 1)
                if (r > s_mid[q + st2 - 1]) q += st2;
            om[i >> 3] = (om[i >> 3] << BM) + q;
        }
    };
    auto quant_m_done = [&]() {
        if constexpr (BM == 2 || M3_FMA) {
            om[0] = (uint32_t)omf[0];
            om[1] = (uint32_t)omf[1];
        }
        if constexpr (M4_FMA) {
            om[0] = (uint32_t)omf4[0] | ((uint32_t)omf4[1] << 16);
            om[1] = (uint32_t)omf4[2] | ((uint32_t)omf4[3] << 16);
        }
        if (dm_new < TINY) { om[0] = 0; om[1] = 0; }             // vanishing block: all codes 0
    };
    if constexpr (!SOLO_F16_MIX) {
        if (!round_m) {
#pragma unroll
            for (int i = EPT16 - 1; i >= 0; --i) quant_m(i);
            quant_m_done();
        }
    }
    if (round_m) {
        // Eq. 5: q = number of levels y_1 .. y_{K-2} that r reaches (the lower end of its bracket), plus
        // one when the element's draw u (Philox purpose 1) falls below (r - y_q) / (y_{q+1} - y_q).
        // "r >= y" is counted on the FMA pipe as the saturation of t - y'*2^100 with t = r*2^100 and y'
        // the binary32 just below y (exactly 0 or 1: two distinct binary32 near a level differ by far
        // more than 2^-100); the level 0 as the saturation of t*2^100 + 1 (t = +-0: 1; else |t*2^100| >=
        // 2^51, or infinite).  NaN counts nowhere and is never below anything: code 0.
        uint32_t wm[8];
        {
            uint32_t ctr_lo, ctr_hi, c3;
            stream_position(ctr_lo, ctr_hi, c3);
            uint32_t w4[4];
            philox_rk(ctr_lo + sw, ctr_hi, a.step32, c3 + 1u, a.rk, w4);
#pragma unroll
            for (int i = 0; i < 4; ++i) wm[i] = w4[i];
            philox_rk(ctr_lo + (sw ^ 1u), ctr_hi, a.step32, c3 + 1u, a.rk, w4);
#pragma unroll
            for (int i = 0; i < 4; ++i) wm[4 + i] = w4[i];
        }
        constexpr int Z = KM / 2 - 1;                             // index of the level 0
        float nb[BM == 4 ? 3 : KM - 2];                           // nb[j - 1]: threshold of level j, BM == 4: of levels 4, 8, 12
        if constexpr (BM == 4) {
            const float4 c4 = s_br[4];
            nb[0] = c4.x; nb[1] = c4.y; nb[2] = c4.z;
        } else {
            const float4 ba = s_br[0];
            nb[0] = ba.x; nb[1] = ba.y;
            if constexpr (BM == 3) {
                const float4 bb = s_br[1];
                nb[2] = ba.z; nb[3] = ba.w; nb[4] = bb.x; nb[5] = bb.y;
            }
        }
        float accm[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int j = EPT16 / 2 - 1; j >= 0; --j) {
            float d[2];                                           // the 16-bit draws of elements 2j, 2j + 1 as binary32
            halves_to_float(wm[j], d[0], d[1]);
#pragma unroll
            for (int e = 1; e >= 0; --e) {
                const int i = 2 * j + e;
                const float r = mh[i] * inv_m;
                const float t = r * BIG;
                float qf;
                if constexpr (BM == 4) {
                    const float c0 = __saturatef(t + nb[0]);
                    const float c1 = __saturatef(t + nb[1]);
                    const float c2 = __saturatef(t + nb[2]);
                    const float o = __fmaf_rn(c2, 16.0f, __fmaf_rn(c1, 16.0f, __fmaf_rn(c0, 16.0f, 8388608.0f)));
                    // row s: thresholds of levels 4s+1, 4s+2, 4s+3 (.w: the factor of t for the third,
                    // 2^100 where that level is 0)
                    const float4 row = *reinterpret_cast<const float4*>(reinterpret_cast<const char*>(s_br) + (__float_as_uint(o) & 0x30u));
                    qf = __fmaf_rn((c0 + c1) + c2, 4.0f, __saturatef(t + row.x));
                    qf += __saturatef(t + row.y);
                    qf += __saturatef(__fmaf_rn(t, row.w, row.z));
                } else {
                    qf = 0.0f;
#pragma unroll
                    for (int l = 1; l <= KM - 2; ++l)
                        qf += l == Z ? __saturatef(__fmaf_rn(t, BIG, 1.0f)) : __saturatef(t + nb[l - 1]);
                }
                // the bracket's lower level and the reciprocal of its width, from the pair table
                const float o8 = __fmaf_rn(qf, 8.0f, 8388608.0f);
                const float2 yg = *reinterpret_cast<const float2*>(reinterpret_cast<const char*>(s_yg) + (__float_as_uint(o8) & 0xF8u));
                const float frac = (r - yg.x) * yg.y;
                const float code = qf + (d[e] < frac * 65536.0f ? 1.0f : 0.0f);     // u = d / 2^16 < frac
                if constexpr (BM == 4) accm[i >> 2] = __fmaf_rn(accm[i >> 2], 16.0f, code);
                else accm[i >> 3] = __fmaf_rn(accm[i >> 3], (float)KM, code);
            }
        }
        if constexpr (BM == 4) {
            om[0] = (uint32_t)accm[0] | ((uint32_t)accm[1] << 16);
            om[1] = (uint32_t)accm[2] | ((uint32_t)accm[3] << 16);
        } else {
            om[0] = (uint32_t)accm[0];
            om[1] = (uint32_t)accm[1];
        }
        if (dm_new < TINY) { om[0] = 0; om[1] = 0; }             // vanishing block: all codes 0
    }

    // ---- (D) second moment: block scale and the p-quantile (k = 13 of 128); the draws of Eq. 6 ----
    mx_v = group_max16<G>(mx_v);
    uint32_t x_p;
    uint32_t w[8];                                                // 16 halfwords: the draws of the 16 elements
    {
        // Philox4x32-10 on the counters of the thread's two groups of eight elements,
        // (ctr, step, 4 * stream) and (ctr + 1, ...), in the thread's order; one round of both per call
        uint32_t ctr_lo, ctr_hi, c3;
        stream_position(ctr_lo, ctr_hi, c3);
        uint32_t ca[4] = {ctr_lo + sw, ctr_hi, a.step32, c3};
        uint32_t cb[4] = {ctr_lo + (sw ^ 1u), ctr_hi, a.step32, c3};
        auto philox_round = [&](int r) {
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                uint32_t(&c)[4] = b ? cb : ca;
                const uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
                const uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
                const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c[1] ^ a.rk[2 * r];
                const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c[3] ^ a.rk[2 * r + 1];
                c[1] = (uint32_t)p1;
                c[3] = (uint32_t)p0;
                c[0] = n0;
                c[2] = n2;
            }
        };
        if (fixed_base) {
            // every block keeps the given base: no quantile to find
            if constexpr (SOLO_F16_MIX) {
                if (!round_m) {
#pragma unroll
                    for (int i = EPT16 - 1; i >= 0; --i) quant_m(i);
                    quant_m_done();
                }
            }
            if (round_v) {
#pragma unroll
                for (int r = 0; r < 10; ++r) philox_round(r);
            }
            x_p = 0u;
        } else {
            uint32_t key[EPT16];
#pragma unroll
            for (int i = 0; i < EPT16; ++i) key[i] = __float_as_uint(vh[i]);
            if (SOLO_F16_MIX && !round_m) {
#pragma unroll
                for (int k = 0; k < 62; ++k) {
                    cswap(key[SORT16_PAIRS[k][0]], key[SORT16_PAIRS[k][1]]);
                    if ((k & 3) == 3 || k == 61) quant_m(15 - (k >> 2));
                }
                quant_m_done();
            } else {
                sort16_low13(key);
            }
            if constexpr (ROUNDS > 12) cswap(key[13], key[14]); // all sixteen in order
            uint32_t* const col = &s.sort[0][tid];
            constexpr int KEPT = ROUNDS < 15 ? ROUNDS : 15;       // keys after the smallest that can be asked for
            // (upper group of sixteen lanes: complemented, see group_min16k)
            const bool hi = G == 16 && (lane & 16);
            const uint32_t vx = hi ? 0xFFFFFFFFu : 0u;
#pragma unroll
            for (int j = 1; j <= KEPT; ++j) col[(j - 1) * CTA16] = key[j] ^ vx;
            // ROUNDS rounds pop the ROUNDS smallest keys of the block, the next minimum is x_p
            const uint32_t self = 1u << lane;
            const uint32_t le = (self | (self - 1u)) & ((G == 32 ? 0xFFFFFFFFu : ((1u << G) - 1u)) << (lane & ~(G - 1)));
            uint32_t head = key[0] ^ vx;
            int off = 0;
#pragma unroll
            for (int r = 0; r < ROUNDS; ++r) {
                pop_round16<G, false, (ROUNDS > 15)>(head, off, col, le, self, hi);
                if (r < 10 && round_v) philox_round(r);
            }
            if (round_v) {
#pragma unroll
                for (int r = ROUNDS; r < 10; ++r) philox_round(r);
            }
            x_p = pop_round16<G, true, false>(head, off, col, le, self, hi) ^ vx;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) { w[i] = ca[i]; w[4 + i] = cb[i]; }
    }

    // ---- (E) per-block scalars by the first warp; the next tile's copies start meanwhile ----
    if (gl == 0) s.xin[grp] = make_uint4(mx_m, mx_v, x_p, 0u);
    bar_sync16(1);
    // every thread has read what it needs from the stage
    if (next_full && tid == 32)
        issue_tile_copy16<BM, BV, PBF, G>(a, s, pt + TILE * PSZ, gt + TILE * 2, jb_tile + NG,
                                       tile_no + 2 == a.debug_stall_tile_p1 ? 16u : 0u);
    if (tid < NG) block_scalars16<KV>(a, s, jb_tile, tid, fixed_base, vtab);
    bar_sync16(2);
    const float4 sc = s.xout[grp];

    // second moment: Eq. 6, see fast_tile
    uint32_t ov[2];
    if (vtab) {
        // Eq. 1 on the fixed codebook: code = number of midpoints below r, counted like the first
        // moment's (saturated multiply-adds, exactly 0 or 1 each: r and a midpoint, if they differ at all,
        // differ by far more than 2^-100, the smallest midpoint of these codebooks being about 1e-4)
        const float inv = sc.y;
        if constexpr (BV <= 3) {
            const float4 na = s_nv[0], nb = s_nv[1];
            float acc[2] = {0.0f, 0.0f};                         // eight codes, at most 24 bits: exact
#pragma unroll
            for (int i = EPT16 - 1; i >= 0; --i) {
                const float r = vh[i] * inv;
                float& c = acc[i >> 3];
                c = __fmaf_rn(c, (float)KV, __saturatef(__fmaf_rn(r, BIG, na.x)));
                c += __saturatef(__fmaf_rn(r, BIG, na.y));
                c += __saturatef(__fmaf_rn(r, BIG, na.z));
                if constexpr (BV == 3) {
                    c += __saturatef(__fmaf_rn(r, BIG, na.w));
                    c += __saturatef(__fmaf_rn(r, BIG, nb.x));
                    c += __saturatef(__fmaf_rn(r, BIG, nb.y));
                    c += __saturatef(__fmaf_rn(r, BIG, nb.z));
                }
            }
            ov[0] = (uint32_t)acc[0];
            ov[1] = (uint32_t)acc[1];
        } else {
            // sixteen levels in two steps of three comparisons, as for 4-bit first moments: row 3 holds
            // the midpoints 3, 7, 11, rows 4..7 the three midpoints inside each quarter
            const float4 nq4 = s_nv[3];
            float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};            // four codes each
#pragma unroll
            for (int i = EPT16 - 1; i >= 0; --i) {
                const float r = vh[i] * inv;
                const float c0 = __saturatef(__fmaf_rn(r, BIG, nq4.x));
                const float c1 = __saturatef(__fmaf_rn(r, BIG, nq4.y));
                const float c2 = __saturatef(__fmaf_rn(r, BIG, nq4.z));
                const float t = __fmaf_rn(c2, 16.0f, __fmaf_rn(c1, 16.0f, __fmaf_rn(c0, 16.0f, 8388608.0f)));
                const float4 row = *reinterpret_cast<const float4*>(reinterpret_cast<const char*>(s_nv + 4) + (__float_as_uint(t) & 0x30u));
                float code = __fmaf_rn((c0 + c1) + c2, 4.0f, __saturatef(__fmaf_rn(r, BIG, row.x)));
                code += __saturatef(__fmaf_rn(r, BIG, row.y));
                code += __saturatef(__fmaf_rn(r, BIG, row.z));
                acc[i >> 2] = __fmaf_rn(acc[i >> 2], 16.0f, code);
            }
            ov[0] = (uint32_t)acc[0] | ((uint32_t)acc[1] << 16);
            ov[1] = (uint32_t)acc[2] | ((uint32_t)acc[3] << 16);
        }
        if (sc.x != 0.0f) { ov[0] = 0; ov[1] = 0; }              // vanishing block: all codes 0
    } else {
        const float inv = sc.y, il = sc.z, lim = sc.w;
        constexpr float KM1 = (float)(KV - 1);
        constexpr float MAGIC = 12582912.0f;
        constexpr uint32_t MAGIC_BITS = 0x4B400000u;
        const float ils = il * (1.0f / KM1);
        // xi = (d + 1/2) / 2^16 - 1/2 (exact), scaled like t; zero without the dither
        const float xs1 = round_v ? (float)(0x1p-16 / (KV - 1)) : 0.0f;
        const float xs0 = round_v ? (float)((-0.5 + 0x1p-17) / (KV - 1)) : 0.0f;
        float worst = 0.0f;
        uint32_t acc[2] = {0u, 0u};
#pragma unroll
        for (int j = EPT16 / 2 - 1; j >= 0; --j) {
            float d[2];                                           // the 16-bit draws of elements 2j, 2j + 1 as binary32
            halves_to_float(w[j], d[0], d[1]);
#pragma unroll
            for (int e = 1; e >= 0; --e) {
                const int i = 2 * j + e;
                const float r = vh[i] * inv;
                const float ts = __saturatef(__fmaf_rn(lg2_approx(r), ils, __fmaf_rn(d[e], xs1, xs0)));
                const float u = __fmaf_rn(ts, KM1, MAGIC);
                worst = fmaxf(worst, fabsf(__fmaf_rn(ts, KM1, MAGIC - u)));
                acc[i >> 3] = acc[i >> 3] * (1u << BV) + __float_as_uint(u);
            }
        }
        uint32_t magic_sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) magic_sum = (magic_sum << BV) + MAGIC_BITS;
        ov[0] = acc[0] - magic_sum;
        ov[1] = acc[1] - magic_sum;
        if (__any_sync(0xffffffffu, worst > lim)) {
            // too close to a rounding boundary for the approximate logarithm somewhere in the warp:
            // the exact sequence for all sixteen
            const float x1 = round_v ? 0x1p-16f : 0.0f, x0 = round_v ? -0.5f + 0x1p-17f : 0.0f;
            ov[0] = 0;
            ov[1] = 0;
#pragma unroll
            for (int j = EPT16 / 2 - 1; j >= 0; --j) {
                float d[2];
                halves_to_float(w[j], d[0], d[1]);
#pragma unroll
                for (int e = 1; e >= 0; --e) {
                    const int i = 2 * j + e;
                    const float r = vh[i] * inv;
                    uint32_t q = KV - 1;
                    if (!(r < TINY)) {
                        float t = __fmaf_rn(log2_sp(r), il, __fmaf_rn(d[e], x1, x0));
                        t = fminf(fmaxf(t, 0.0f), KM1);
                        q = (uint32_t)__float2int_rn(t);
                    }
                    ov[i >> 3] = (ov[i >> 3] << BV) + q;
                }
            }
        }
        if (sc.x != 0.0f) { ov[0] = 0; ov[1] = 0; }              // vanishing block: all codes 0
    }

    // ---- store the codes ----
    const uint32_t om_e[2] = {sw ? om[1] : om[0], sw ? om[0] : om[1]};      // back to element order
    const uint32_t ov_e[2] = {sw ? ov[1] : ov[0], sw ? ov[0] : ov[1]};
    store_codes16<BM>(a.codes_m + jb_tile * (2 * G * BM), s.cout[0][BM == 3 ? warp : 0], tid, om_e);
    store_codes16<BV>(a.codes_v + jb_tile * (2 * G * BV), s.cout[(BM == 3 && BV == 3) ? 1 : 0][BV == 3 ? warp : 0], tid, ov_e);
}

template <int BM, int BV, bool PBF, int G, int MODES>
__global__ void __launch_bounds__(CTA16, SOLO_F16_CTAS) solo_step_fast16_kernel(const StepArgs a) {
    constexpr int KM = 1 << BM;
    constexpr bool EXT = MODES == 2;
    using Shared = Fast16Shared<BM, BV, PBF, G>;
    extern __shared__ __align__(16) unsigned char fast16_smem[];
    Shared& s = *reinterpret_cast<Shared*>(fast16_smem);
    __shared__ float s_y[KM];
    __shared__ float s_mid[KM];
    __shared__ float2 s_yg[EXT ? KM : 1];                    // Eq. 5: see the set-up below
    __shared__ float4 s_br[EXT ? (BM == 4 ? 5 : 2) : 1];
    __shared__ float s_yv[EXT ? 1 << BV : 1];               // baseline second-moment codebook: its levels,
    __shared__ float4 s_nv[EXT ? 8 : 1];                     // its midpoints times -2^100 (rows as the tile function reads them)
    __shared__ float4 s_mid4[4];             // 4-bit first moments: per quarter of the codebook, its three inner midpoints times -2^100
    const int tid = threadIdx.x;
    if (tid < KM) {
        s_y[tid] = a.tables[tid];
        if (tid < KM - 1) s_mid[tid] = a.tables[KM + tid];
    }
    if (BM == 4 && tid < 4)
        s_mid4[tid] = make_float4(-a.tables[KM + 4 * tid] * 0x1p100f, -a.tables[KM + 4 * tid + 1] * 0x1p100f,
                                  -a.tables[KM + 4 * tid + 2] * 0x1p100f, 0.0f);
    if constexpr (EXT) {
        if (a.round_m) {
            // Eq. 5: per level q <= K-2 the pair (y_q, 1 / (y_{q+1} - y_q)); thresholds of "r >= y_j" as
            // -y'_j * 2^100, y'_j the binary32 just below y_j (rows as the tile function reads them:
            // 2- and 3-bit, levels 1..6 in rows 0, 1; 4-bit, row s = levels 4s+1..4s+3 and row 4 = levels
            // 4, 8, 12).  The level 0 is compared another way; a level past K-2 gets -infinity: never reached.
            const float* const yk = a.tables;
            auto below = [&](int j) {
                const float y = yk[j];
                return -__uint_as_float(__float_as_uint(y) + (y < 0.0f ? 1u : 0xFFFFFFFFu)) * 0x1p100f;
            };
            if (tid < KM - 1) s_yg[tid] = make_float2(yk[tid], a.tables[2 * KM - 1 + tid]);
            if (BM <= 3 && tid < 2) {
                float t4[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int j = 4 * tid + k + 1;
                    t4[k] = j <= KM - 2 && j != KM / 2 - 1 ? below(j) : 0.0f;
                }
                s_br[tid] = make_float4(t4[0], t4[1], t4[2], t4[3]);
            }
            if (BM == 4 && tid < 4) {
                const int j = 4 * tid + 1;
                const bool zero3 = j + 2 == KM / 2 - 1;            // the row's third level is the level 0
                s_br[tid] = make_float4(below(j), below(j + 1),
                                        zero3 ? 1.0f : j + 2 <= KM - 2 ? below(j + 2) : -__int_as_float(0x7f800000),
                                        zero3 ? 0x1p100f : 1.0f);
            }
            if (BM == 4 && tid == 4) s_br[4] = make_float4(below(4), below(8), below(12), 0.0f);
        }
        if (a.tables_v != nullptr) {
            constexpr int KV = 1 << BV;
            const float* const midv = a.tables_v + KV;            // KV - 1 midpoints
            if (tid < KV) s_yv[tid] = a.tables_v[tid];
            if (tid < 2) {                                         // rows 0, 1: midpoints 0..7 (rows of 3 or 7 are padded)
                float m4[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) m4[k] = 4 * tid + k < KV - 1 ? -midv[4 * tid + k] * 0x1p100f : 0.0f;
                s_nv[tid] = make_float4(m4[0], m4[1], m4[2], m4[3]);
            }
            if (BV == 4 && tid == 3)
                s_nv[3] = make_float4(-midv[3] * 0x1p100f, -midv[7] * 0x1p100f, -midv[11] * 0x1p100f, 0.0f);
            if (BV == 4 && tid >= 4 && tid < 8)
                s_nv[tid] = make_float4(-midv[4 * (tid - 4)] * 0x1p100f, -midv[4 * (tid - 4) + 1] * 0x1p100f,
                                        -midv[4 * (tid - 4) + 2] * 0x1p100f, 0.0f);
        }
    }
    // (never overwritten: rows 0..14 hold keys; complemented for the upper group of sixteen lanes)
    if constexpr (Shared::ROWS == 16) s.sort[15][tid] = (G == 16 && (tid & 16)) ? ~KEY_MAX : KEY_MAX;
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s.mbar)) : "memory");
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
    Ahead16 ah;
    const bool decay = a.decay != 1.0f;
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
        const bool next_full = tin + 1 < full_tiles && tile + 1 < tile_end;
        if (decay)
            fast16_tile<BM, BV, PBF, G, true, MODES>(a, s, s_y, s_mid, s_mid4, s_yv, s_nv, s_yg, s_br, pbase, gbase, tin, jb0 + (int64_t)tin * Shared::NG, tensor, ah, next_full, tile);
        else
            fast16_tile<BM, BV, PBF, G, false, MODES>(a, s, s_y, s_mid, s_mid4, s_yv, s_nv, s_yg, s_br, pbase, gbase, tin, jb0 + (int64_t)tin * Shared::NG, tensor, ah, next_full, tile);
    }
    // A thread that gave up on a copy waits once more, again bounded, for the last one that was issued,
    // so that no copy is still writing to the stage when the CTA's shared memory is released.
    if (ah.failed && ah.fill > 0) mbar_wait(smem_u32(&s.mbar), (ah.fill - 1u) & 1u);
}

}  // namespace solo
