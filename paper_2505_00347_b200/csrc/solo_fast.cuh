// Streamlined fused step for the common configurations: 2/3/4/8-bit states, blocks of
// 64, 128, 256 or 2048 elements, fp32 or bf16 parameters, the paper's logarithmic quantizer for the
// second moment, nearest rounding of the first moment, eps >= 1e-12.
//
// Same packed state as the general kernel (solo_device.cuh): every quantity that decides
// a stored code (EMA values, block scales, p-quantile, base, rounded logarithm) is computed
// with the same IEEE operation sequence or is proven equal to it:
//   * log_alpha(r) + xi is first evaluated with the hardware lg2 approximation; only when
//     the result lies within a proven error bound of a rounding boundary is the exact
//     polynomial log2_sp evaluated (rare), so the rounded code is always the one the exact
//     sequence gives;
//   * the k-th smallest v^ of a block is found exactly, duplicates included, by popping one
//     minimum per round from per-thread sorted lists.
// The update of fp32 parameters uses an approximate square root and a reciprocal refined by
// one Newton step (quotient error below 1.5 ulp); they therefore agree with the IEEE sequence
// to a few 1e-7 of the update term, not bit for bit.  bf16 parameters (PBF) are rounded from
// the binary32 result, where such a difference could flip a whole bf16 ulp: that variant uses
// the IEEE square root and division and stores the same patterns as the general kernel.
//
// Work split: a CTA of 256 threads owns a tile of 2048 consecutive elements, a thread
// eight of them, a block of B elements G = B/8 consecutive lanes (a quarter, half or whole warp;
// G = 256: the whole CTA, with CTA-wide maxima and a radix select instead of the warp collectives).
// The per-block scalar work (reciprocals of the scales, base of the logarithmic codebook
// and its logarithm) is done once per block by the first warp for the whole tile and
// passed through shared memory.
//
// Warp collectives are always issued with the full mask (one REDUX each).  For G = 16 the
// two halves of a warp are reduced by one minimum and one maximum over a transformed
// value: all quantities reduced here are non-negative binary32 bit patterns (bit 31
// clear), so complementing the upper half's values moves them above every lower-half
// value and reverses their order.  For G = 8 (four groups per warp) three shuffle-and-compare
// steps over the untransformed values serve all groups at once.
#pragma once

#include <type_traits>

#include "solo_device.cuh"

namespace solo {

// Error model of lg2.approx.ftz.f32 against log2_sp, |diff| <= LG2_ABS + LG2_REL * |log2 x|
// (checked exhaustively over all binary32 in [2^-100, 2) by solo_debug_check_fast_log with
// half of these constants); the other half of LG2_REL covers the roundings of t, which the
// kernel evaluates scaled to [0, 1] (a few 2^-24 relative each).
constexpr float LG2_ABS = 0x1p-20f;
constexpr float LG2_REL = 0x1p-20f;

constexpr uint32_t KEY_MAX = 0x7FFFFFFFu;    // sentinel key: above or equal to every valid key

// WM, WV: 32-bit words of packed codes per thread (1 up to 4-bit codes, 2 for 8-bit codes).
template <int WM, int WV>
struct FastSharedT {
    uint32_t sort[16][CTA];                  // rows 0..6: 2nd..8th smallest key of a thread; rows 7..15: sentinel
    float tab[CTA / 8][32];                 // per group: second-moment levels (8-bit: alpha^0..15), then K_m
                                            // first-moment levels (8-bit first moments use the codebook itself)
    uint4 xin[2][CTA / 8];                  // per group: bits of Delta_m', Delta_v', x_p
    float4 xout[2][CTA / 8];                // per group: 1/Delta_m', 1/Delta_v', 1/log2(alpha'), rounding limit
    uint32_t xflag[2][CTA / 8];             // bit 0: vanishing first moment, bit 1: vanishing second moment
    uint32_t red[2][24];                    // G = 256: per-warp maxima of |m^| (0..7) and v^ (8..15), minima of v^ (16..23)
    // Two stages for the inputs of a full tile, filled by bulk asynchronous copies (TMA, issued by
    // one thread) one tile ahead of their use; each stage has its own mbarrier.
    struct Stage {
        float4 p[2 * CTA];                   // 2048 parameters (bf16: the first half)
        uint4 g[CTA];                        // 2048 bf16 gradients
        uint32_t cm[WM * CTA + 4];           // packed codes of the tile, from a 16-byte boundary (64 * bits words + 2)
        uint32_t cv[WV * CTA + 4];
        float sc[3][CTA / 8 + 4];            // Delta_m, Delta_v, alpha of the tile's blocks, from a 16-byte boundary
    };
    alignas(16) Stage stage[2];
    alignas(8) unsigned long long mbar[2];
};
template <int BM, int BV>
using FastShared = FastSharedT<(BM == 8 ? 2 : 1), (BV == 8 ? 2 : 1)>;

// What a CTA carries from one tile to the next for the copy-ahead of inputs.
struct Ahead {
    uint32_t fill = 0;        // number of the next bulk copy to wait for (uniform over the CTA)
    bool staged = false;      // that copy has already been issued (uniform)
    bool failed = false;      // this thread once waited in vain for a copy: it polls once per tile from then on
                              // and its warp stores nothing
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Waits until the phase with the given parity of an mbarrier has completed.  Bounded: gives up
// (returns false) after `polls` timed-out polls (2^14 unless told otherwise) instead of spinning for ever.
constexpr int MBAR_POLLS = 1 << 14;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int polls = MBAR_POLLS) {
    for (int it = 0; it < polls; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void bulk_copy(void* smem_dst, const void* gmem_src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ float lg2_approx(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float sqrt_approx(float x) {
    float y;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// max(acc, |x|) that returns NaN when x is NaN: a NaN among the block's values makes the block's
// scale NaN, as the maximum over bit patterns of the general kernel does.
__device__ __forceinline__ float max_abs_nan(float acc, float x) {
    float r;
    asm("{\n\t.reg .f32 t;\n\tabs.f32 t, %2;\n\tmax.NaN.f32 %0, %1, t;\n\t}" : "=f"(r) : "f"(acc), "f"(x));
    return r;
}

// The two 16-bit halves of a word as binary32 (one conversion each, no shift or mask).
__device__ __forceinline__ void halves_to_float(uint32_t w, float& lo, float& hi) {
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.rn.f32.u16 %0, l;\n\tcvt.rn.f32.u16 %1, h;\n\t}"
        : "=f"(lo), "=f"(hi) : "r"(w));
}

// Byte offsets (4 * code) of the eight W-bit codes packed in `c`, for a table of floats.  The
// codes at even and at odd positions are kept in two words with the other positions zeroed, so
// that a left shift that brings a code to the top of the word followed by a right shift leaves
// 4 * code without a mask.
template <int W>
struct CodeOffsets {
    uint32_t even, odd;
    __device__ __forceinline__ CodeOffsets(uint32_t c, uint32_t) {
        uint32_t me = 0;
#pragma unroll
        for (int i = 0; i < 8; i += 2) me |= ((1u << W) - 1u) << (i * W);
        even = c & me;
        odd = c & (me << W);
    }
    __device__ __forceinline__ uint32_t operator()(int i) const {
        const uint32_t w = (i & 1) ? odd : even;
        uint32_t top;       // the code moved to the top of the word (a multiply: kept apart from the shift)
        asm("mul.lo.u32 %0, %1, %2;" : "=r"(top) : "r"(w), "r"(1u << (32 - (i + 1) * W)));
        return top >> (30 - W);
    }
};

// 8-bit codes: four per word (`lo`: elements 0..3, `hi`: elements 4..7); a byte is brought to
// bits 2..9 by one shift and masked.  low4(i): byte offset of entry (code & 15) of a table of
// floats; bit(i, k): bit k of the code.
template <>
struct CodeOffsets<8> {
    uint32_t lo, hi;
    __device__ __forceinline__ CodeOffsets(uint32_t l, uint32_t h) : lo(l), hi(h) {}
    __device__ __forceinline__ uint32_t word(int i) const { return i < 4 ? lo : hi; }
    __device__ __forceinline__ uint32_t operator()(int i) const {
        const int j = i & 3;
        return j == 0 ? (word(i) << 2) & 0x3FCu : (word(i) >> (8 * j - 2)) & 0x3FCu;
    }
    __device__ __forceinline__ uint32_t low4(int i) const {
        const int j = i & 3;
        return j == 0 ? (word(i) << 2) & 0x3Cu : (word(i) >> (8 * j - 2)) & 0x3Cu;
    }
    __device__ __forceinline__ bool bit(int i, int k) const { return ((word(i) >> (8 * (i & 3) + k)) & 1u) != 0; }
};

// Philox4x32-10 with the round keys taken from the kernel arguments.
__device__ __forceinline__ void philox_rk(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                          const uint32_t (&rk)[20], uint32_t (&out)[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ rk[2 * r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ rk[2 * r + 1];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// ---------------------------------------------------------------------------
// Group collectives on 31-bit values.
// `hi` (G = 16 only): the lane belongs to the upper half of the warp, the odd group of the pair.
// ---------------------------------------------------------------------------

// min over the even group and max over the odd group of `u`, for the calling lane's pair; returns
// the one that belongs to the lane's own group
template <int G>
__device__ __forceinline__ uint32_t seg_pick(uint32_t u, bool hi) {
    static_assert(G == 16, "two groups of sixteen lanes");
    const uint32_t lo = __reduce_min_sync(0xffffffffu, u);
    const uint32_t up = __reduce_max_sync(0xffffffffu, u);
    return hi ? up : lo;
}
template <int G>
__device__ __forceinline__ uint32_t seg_max31(uint32_t x, bool hi) {
    if constexpr (G == 32) {
        return __reduce_max_sync(0xffffffffu, x);
    } else if constexpr (G == 8) {
        // four groups per warp: three shuffle-and-compare steps serve them all and were measured
        // faster than four reductions plus selects (the groups of eight use no transformed domain:
        // `hi` is false for them)
#pragma unroll
        for (int d = 1; d < 8; d <<= 1) x = max(x, __shfl_xor_sync(0xffffffffu, x, d));
        return x;
    } else {
        // even group: complement of the low 31 bits (order reversed, bit 31 clear); odd group:
        // bit 31 set.  min = even group's maximum, max = odd group's maximum.
        const uint32_t c = hi ? 0x80000000u : 0x7FFFFFFFu;
        return seg_pick<G>(x ^ c, hi) ^ c;
    }
}
// Minimum of the group's keys in the "v domain": even group keeps x, odd group holds ~x.
// Returns the value a lane compares its own v with (equal <=> the lane holds the minimum).
template <int G>
__device__ __forceinline__ uint32_t seg_min_v(uint32_t v, bool hi) {
    if constexpr (G == 32) {
        return __reduce_min_sync(0xffffffffu, v);
    } else if constexpr (G == 8) {
#pragma unroll
        for (int d = 1; d < 8; d <<= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, d));
        return v;
    } else {
        return seg_pick<G>(v, hi);
    }
}

// Codes of the thread's eight elements.  2 and 4 bit: one aligned 16/32-bit access.
// 3 bit: the warp's 256 codes are 24 consecutive words; lanes 0..23 access one word
// each and the 24-bit pieces travel by shuffle.
template <int BITS>
__device__ __forceinline__ uint32_t warp_load_codes(const uint8_t* warp_base, int lane) {
    if constexpr (BITS == 2) {
        return __ldcs(reinterpret_cast<const unsigned short*>(warp_base) + lane);
    } else if constexpr (BITS == 4) {
        return __ldcs(reinterpret_cast<const unsigned int*>(warp_base) + lane);
    } else {
        uint32_t w = 0;
        if (lane < 24) w = __ldcs(reinterpret_cast<const unsigned int*>(warp_base) + lane);
        const int a = (3 * lane) >> 2, o = ((3 * lane) & 3) * 8;
        const uint32_t lo = __shfl_sync(0xffffffffu, w, a);
        const uint32_t hi = __shfl_sync(0xffffffffu, w, (a + 1) & 31);
        return __funnelshift_r(lo, hi, o) & 0xFFFFFFu;
    }
}
// Issues (one thread) the bulk copies of one full tile's inputs into stage `fill & 1`: parameters,
// gradients, the packed codes of its blocks and their three per-block scalars.  Bulk copies need
// 16-byte aligned addresses and sizes: codes (8 bytes off for 3-bit codes in blocks of 64 when the
// first block is odd) and scalars are copied from the 16-byte boundary at or below them, with 16
// bytes more when they do not start on it; readers add the offset.  The scalar arrays are
// allocated in multiples of 16 bytes, so the copy never leaves them.
// `extra_tx`: bytes announced on top of what is copied (test hook: the wait for this tile then runs out).
template <int BM, int BV, int G, bool PBF>
__device__ __forceinline__ void issue_tile_copy(const StepArgs& a, FastShared<BM, BV>& s, uint32_t fill, const char* pt,
                                                const char* gt, int64_t jb_tile, uint32_t extra_tx) {
    constexpr int NG = CTA / G;
    constexpr uint32_t PBYTES = TILE * (PBF ? 2 : 4);
    typename FastShared<BM, BV>::Stage& st = s.stage[fill & 1u];
    const uint32_t bar = smem_u32(&s.mbar[fill & 1u]);
    const int64_t bm0 = jb_tile * G * BM, bv0 = jb_tile * G * BV;   // byte offsets of the tile's codes
    const uint32_t bytes_m = CTA * BM + ((bm0 & 15) ? 16u : 0u), bytes_v = CTA * BV + ((bv0 & 15) ? 16u : 0u);
    // NG >= 8 scalars from the boundary below the first (16 bytes more when it is not on it); a
    // single block's scalar (NG = 1) lies within the 16 bytes that start at that boundary
    const uint32_t bytes_s = NG >= 4 ? (NG + ((jb_tile & 3) ? 4u : 0u)) * 4u : 16u;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar),
                 "r"((uint32_t)(PBYTES + TILE * 2) + bytes_m + bytes_v + 3u * bytes_s + extra_tx) : "memory");
    bulk_copy(st.p, pt, PBYTES, bar);
    bulk_copy(st.g, gt, TILE * 2, bar);
    bulk_copy(st.cm, a.codes_m + (bm0 & ~(int64_t)15), bytes_m, bar);
    bulk_copy(st.cv, a.codes_v + (bv0 & ~(int64_t)15), bytes_v, bar);
    const int64_t j0 = jb_tile & ~(int64_t)3;
    bulk_copy(st.sc[0], a.scale_m + j0, bytes_s, bar);
    bulk_copy(st.sc[1], a.scale_v + j0, bytes_s, bar);
    bulk_copy(st.sc[2], a.alpha + j0, bytes_s, bar);
}

// From the warp's packed words (lane < 24 holds word `lane`) to the thread's own 3-bit codes.
template <int BITS>
__device__ __forceinline__ uint32_t warp_codes_finish(uint32_t w, int lane) {
    static_assert(BITS == 3, "only the 3-bit layout needs the exchange");
    const int a = (3 * lane) >> 2, o = ((3 * lane) & 3) * 8;
    const uint32_t lo = __shfl_sync(0xffffffffu, w, a);
    const uint32_t hi = __shfl_sync(0xffffffffu, w, (a + 1) & 31);
    return __funnelshift_r(lo, hi, o) & 0xFFFFFFu;
}
template <int BITS>
__device__ __forceinline__ void warp_store_codes(uint8_t* warp_base, int lane, uint32_t c) {
    if constexpr (BITS == 2) {
        __stcs(reinterpret_cast<unsigned short*>(warp_base) + lane, (unsigned short)c);
    } else if constexpr (BITS == 4) {
        __stcs(reinterpret_cast<unsigned int*>(warp_base) + lane, c);
    } else {
        const int a = (4 * lane) / 3, o = 32 * lane - 24 * a;        // o in {0, 8, 16} for lane < 24
        const uint32_t lo = __shfl_sync(0xffffffffu, c, a & 31);
        const uint32_t hi = __shfl_sync(0xffffffffu, c, (a + 1) & 31);
        if (lane < 24)
            __stcs(reinterpret_cast<unsigned int*>(warp_base) + lane, (lo >> (o & 31)) | (hi << ((24 - o) & 31)));
    }
}

__device__ __forceinline__ void sort8(uint32_t (&key)[EPT]) {
    cswap(key[0], key[1]); cswap(key[2], key[3]); cswap(key[4], key[5]); cswap(key[6], key[7]);
    cswap(key[0], key[2]); cswap(key[1], key[3]); cswap(key[4], key[6]); cswap(key[5], key[7]);
    cswap(key[1], key[2]); cswap(key[5], key[6]); cswap(key[0], key[4]); cswap(key[3], key[7]);
    cswap(key[1], key[5]); cswap(key[2], key[6]);
    cswap(key[1], key[4]); cswap(key[3], key[6]);
    cswap(key[2], key[4]); cswap(key[3], key[5]);
    cswap(key[3], key[4]);
}

// One selection round: finds the group's smallest unpopped key and pops it from exactly one
// thread (the lowest lane among those whose head equals it), so that after r rounds the r
// smallest keys, duplicates included, have been popped.  Returns that key (v domain).
// `off` is the word offset of the thread's next row in its column `col`, `le` the mask of the
// lanes of the thread's group up to and including it, `self` the thread's own lane bit.
// Unclamped form: `off` advances one row per pop and may be used for at most 16 rounds (rows
// 7..15 of a column hold the sentinel).  Clamped form: any number of rounds; the offset stops at
// the first sentinel row.
template <int G, bool CLAMP, bool LAST = false>
__device__ __forceinline__ uint32_t pop_round(uint32_t& head, int& off, const uint32_t* col, uint32_t le,
                                              uint32_t self, bool hi) {
    if constexpr (LAST) return seg_min_v<G>(head, hi);          // the answer; nothing left to pop
    const uint32_t nxt = col[off];                               // the key that follows, should this thread pop
    const uint32_t tgt = seg_min_v<G>(head, hi);
    // the lowest lane of the group whose head equals the minimum pops: its own bit is the lowest
    // set bit of the ballot within the lanes of its group up to itself
    const uint32_t upto = __ballot_sync(0xffffffffu, head == tgt) & le;
    // if (upto == self) { head = nxt; off += CTA; }  as two predicated instructions
    asm("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, %2, %3;\n\t@p mov.u32 %0, %4;\n\t@p add.s32 %1, %1, %5;\n\t}"
        : "+r"(head), "+r"(off) : "r"(upto), "r"(self), "r"(nxt), "n"(CTA));
    if constexpr (CLAMP) off = min(off, 7 * CTA);
    return tgt;
}

// k-th smallest key of the group (duplicates counted), v domain.  k is uniform over the group
// and may differ between the two halves of a warp (k <= 0: a group without a block, result
// unused).  `col` is the thread's column of sorted keys (rows 0..6, sentinels from row 7 on),
// `head` its smallest key.  UNIFORM_K: every group of the warp has the same k.
// `side(i)`, i = 0..7, is independent work of the caller (the parameter update of element i)
// that is issued between the rounds, where the warp would otherwise wait for the collectives.
template <int G, bool UNIFORM_K, class Side>
__device__ __forceinline__ uint32_t select_kth(uint32_t head, const uint32_t* col, int k, bool hi, Side&& side) {
    const int lane = threadIdx.x & 31;
    const uint32_t self = 1u << lane;
    const uint32_t upto = self | (self - 1u);
    const uint32_t le = G == 32 ? upto : upto & (((1u << G) - 1u) << (lane & ~(G - 1)));
    int off = 0;
    uint32_t ans = 0;
    if (UNIFORM_K && k == 13) {                                  // p = 0.1, block 128
#pragma unroll
        for (int r = 0; r < 12; ++r) {
            pop_round<G, false>(head, off, col, le, self, hi);
            if (r < EPT) side(r);
        }
        ans = pop_round<G, false, true>(head, off, col, le, self, hi);
    } else if (UNIFORM_K && G == 32 && k == 26) {               // p = 0.1, block 256
#pragma unroll
        for (int r = 0; r < 25; ++r) {
            pop_round<G, true>(head, off, col, le, self, hi);
            if (r < EPT) side(r);
        }
        ans = pop_round<G, true, true>(head, off, col, le, self, hi);
    } else if (UNIFORM_K && k == 7) {                            // p = 0.1, block 64
#pragma unroll
        for (int r = 0; r < 6; ++r) {
            pop_round<G, false>(head, off, col, le, self, hi);
            side(r);
        }
        side(6);
        side(7);
        ans = pop_round<G, false, true>(head, off, col, le, self, hi);
    } else {
#pragma unroll
        for (int i = 0; i < EPT; ++i) side(i);
        const int rounds = UNIFORM_K ? k : __reduce_max_sync(0xffffffffu, k);
        if (rounds <= 16) {
#pragma unroll 1
            for (int r = 1; r <= rounds; ++r) {
                const uint32_t t = pop_round<G, false>(head, off, col, le, self, hi);
                if (r == k) ans = t;
            }
        } else {
#pragma unroll 1
            for (int r = 1; r <= rounds; ++r) {
                const uint32_t t = pop_round<G, true>(head, off, col, le, self, hi);
                if (r == k) ans = t;
            }
        }
    }
    return ans;
}

// k-th smallest (1-based, duplicates counted) of the CTA's 2048 keys, eight per thread.  Keys are
// below 2^31, or the all-ones filler of elements that do not exist (k never reaches those); `lo` and
// `hi` are the smallest and the largest key that exists.
// Radix select from the top over the bits of key - lo that can be set (those of hi - lo), eleven at a
// time with 2048 histogram bins (eight per thread): the first level spreads the block's own range of
// values over all bins, whatever its position and width on the number line (the top bits of the keys
// themselves, sign and exponent, would put a block's values into a few dozen bins).  As soon as the bin
// that holds the rank has at most 32 keys, those are collected and ranked directly by the first warp,
// which is the usual case after the first level.  Exact for any input: with many equal keys the levels
// run on until every bit is fixed.  `hist` is 2096 words of shared memory.  Every thread of the CTA calls
// it with the same k, lo and hi; all return the same key.
__device__ __forceinline__ uint32_t cta_select(const uint32_t (&key)[EPT], int k, uint32_t* hist, uint32_t lo,
                                               uint32_t hi) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t* const scan = hist + 2048;      // [0..7] warp totals, [8] bin, [9] rank in it, [10] its count,
                                             // [11] fill of `list`, [12] the answer
    uint32_t* const list = hist + 2048 + 16; // the keys of a bin with at most 32 of them
    if (hi == lo) return lo;                 // (uniform) every key that exists is the same
    int remaining = 32 - __clz(hi - lo);     // bits of key - lo not fixed yet: at most 31
    uint32_t prefix = 0, kk = (uint32_t)k;
#pragma unroll 1
    for (;;) {
        const int width = min(remaining, 11);
        const int shift = remaining - width;
        __syncthreads();                       // the bins, scan[] and list[] of earlier use are read
        reinterpret_cast<uint4*>(hist)[2 * tid] = make_uint4(0u, 0u, 0u, 0u);
        reinterpret_cast<uint4*>(hist)[2 * tid + 1] = make_uint4(0u, 0u, 0u, 0u);
        if (tid == 0) scan[11] = 0;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < EPT; ++i) {       // (the filler minus lo is at least 2^31: it matches no prefix)
            const uint32_t d = key[i] - lo;
            if ((d >> remaining) == prefix) atomicAdd(&hist[(d >> shift) & ((1u << width) - 1u)], 1u);
        }
        __syncthreads();
        const uint4 c0 = reinterpret_cast<const uint4*>(hist)[2 * tid];
        const uint4 c1 = reinterpret_cast<const uint4*>(hist)[2 * tid + 1];
        const uint32_t c[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
        uint32_t mine = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) mine += c[j];
        uint32_t incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += t;
        }
        if (lane == 31) scan[warp] = incl;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < 7; ++w)
            if (w < warp) incl += scan[w];
        uint32_t run = incl - mine;            // keys in the bins before this thread's
        if (kk > run && kk <= incl) {          // exactly one thread holds the rank
            int sel = 0;
            uint32_t cnt = c[0];
#pragma unroll
            for (int j = 0; j < 7; ++j)
                if (kk > run + c[j] && sel == j) {
                    run += c[j];
                    sel = j + 1;
                    cnt = c[j + 1];
                }
            scan[8] = 8u * (uint32_t)tid + (uint32_t)sel;
            scan[9] = kk - run;
            scan[10] = cnt;
        }
        __syncthreads();
        prefix = (prefix << width) | scan[8];
        kk = scan[9];
        const uint32_t cnt = scan[10];
        remaining = shift;
        if (remaining == 0) break;             // every bit is fixed
        if (cnt <= 32u) {                      // uniform: rank the bin's keys directly
#pragma unroll
            for (int i = 0; i < EPT; ++i)
                if (((key[i] - lo) >> remaining) == prefix) list[atomicAdd(&scan[11], 1u)] = key[i];
            __syncthreads();
            if (warp == 0) {
                const uint32_t my = (uint32_t)lane < cnt ? list[lane] : 0xFFFFFFFFu;
                uint32_t below = 0;
                for (uint32_t j = 0; j < cnt; ++j) {
                    const uint32_t o = list[j];
                    below += (o < my || (o == my && j < (uint32_t)lane)) ? 1u : 0u;
                }
                if ((uint32_t)lane < cnt && below == kk - 1u) scan[12] = my;
            }
            __syncthreads();
            return scan[12];
        }
    }
    return lo + prefix;
}

__device__ __forceinline__ void bar_sync(int id) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(CTA) : "memory");
}

// One tile.  FULL: all 2048 elements exist and both tensor pointers are 16-byte aligned; its
// inputs come from a shared-memory stage that bulk asynchronous copies filled while the tile
// before it was worked on (per-thread cp.async staging, L2 prefetch and register prefetch of the
// next tile were all measured slower than plain 128-bit loads; the bulk copies, issued by one
// thread, are faster).  Other tiles (tails, unaligned tensors) use masked plain loads.
// `par` alternates between tiles (double buffering of the per-block exchange arrays); `ah`
// carries the copy-ahead state; next_full / next_dtin describe the CTA's next tile.
template <int BM, int BV, int G, bool FULL, bool PBF, bool PLAIN>
__device__ __forceinline__ void fast_tile(const StepArgs& a, FastShared<BM, BV>& s, const float* s_y,
                                          const float* s_mid, const float4* s_mid4, char* pbase, const char* gbase,
                                          const int64_t n, const int tin, const int64_t jb_tile,
                                          const int tensor, const int par, Ahead& ah, const bool next_full,
                                          const int next_dtin, const int64_t tile_no) {
    constexpr int KM = 1 << BM, KV = 1 << BV;
    constexpr int NG = CTA / G, B = G * EPT;
    constexpr int PSZ = PBF ? 2 : 4;                            // bytes per parameter
    // PLAIN: the step of the paper as it stands (Adam(W) without an L2 term in the gradient, base
    // from the p-quantile, xi drawn); the other modes cost branches and argument loads per tile
    const bool l2 = !PLAIN && a.l2, belief = !PLAIN && a.belief;
    const bool fixed_base = !PLAIN && a.fixed_alpha > 0.0f;
    const bool round_v = PLAIN || a.round_v;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gl = tid & (G - 1), grp = tid / G;
    const bool hi = G == 16 && (lane & G) != 0;                 // odd group of its pair (groups of 16 only)
    const uint32_t vflip = hi ? 0xFFFFFFFFu : 0u;               // x domain <-> v domain

    // validity (all true in a full tile)
    const int64_t tile_elem0 = (int64_t)tin * TILE;
    const int64_t rem_tile = n - tile_elem0;                    // elements of the tensor from the tile's first on, > 0
    const bool have_block = FULL || (int64_t)grp * B < rem_tile;
    const int nb = FULL ? B : (int)max((int64_t)0, min((int64_t)B, rem_tile - (int64_t)grp * B));
    const int nv = FULL ? EPT : (int)max((int64_t)0, min((int64_t)EPT, rem_tile - (int64_t)tid * EPT));

    char* const pt = pbase + tile_elem0 * PSZ;                  // the tile's parameters and gradients
    const char* const gt = gbase + tile_elem0 * 2;
    const int64_t tile_slot0 = jb_tile * G;                     // slot = 8 elements = one thread's codes
    const int64_t jb = jb_tile + grp;

    uint8_t* const wcm = a.codes_m + (tile_slot0 + warp * 32) * BM;   // the warp's 32 slots
    uint8_t* const wcv = a.codes_v + (tile_slot0 + warp * 32) * BV;

    // ---- inputs ----
    float p[EPT], g[EPT];
    uint32_t cm = 0, cv = 0, cm_hi = 0, cv_hi = 0;                // *_hi: elements 4..7 of 8-bit codes
    float dm = 0.0f, dv = 0.0f, al = 0.5f;
    if (FULL) {
        // Every full tile reads its inputs from a stage.  Copy number f uses stage f & 1 and
        // completes phase f >> 1 of that stage's mbarrier.  The copy for this tile was issued
        // while the tile before it was worked on (ah.staged), or is issued now (first full tile
        // after a tensor change); the copy for the next tile is issued here.  Before a stage is
        // refilled all threads have finished reading it: they read at the start of a tile and
        // pass that tile's barriers before any thread starts the next one.
        if (tid == 0) {
            if (!ah.staged)
                issue_tile_copy<BM, BV, G, PBF>(a, s, ah.fill, pt, gt, jb_tile, tile_no + 1 == a.debug_stall_tile_p1 ? 16u : 0u);
            if (next_full)
                issue_tile_copy<BM, BV, G, PBF>(a, s, ah.fill + 1u, pt + (int64_t)next_dtin * (TILE * PSZ),
                                           gt + (int64_t)next_dtin * (TILE * 2), jb_tile + (int64_t)next_dtin * NG,
                                           tile_no + next_dtin + 1 == a.debug_stall_tile_p1 ? 16u : 0u);
        }
        const uint32_t mine = ah.fill;
        ah.fill += 1u;
        ah.staged = next_full;
        if (!mbar_wait(smem_u32(&s.mbar[mine & 1u]), (mine >> 1) & 1u, ah.failed ? 1 : MBAR_POLLS)) {
            // the copy was never seen to arrive: flag it (solo_state_status reports bit 1); what the
            // warp then leaves the tile alone (below)
            if (!ah.failed) atomicOr(a.status, 2);
            ah.failed = true;
        }
        const typename FastShared<BM, BV>::Stage& st = s.stage[mine & 1u];
        const uint4 gw = st.g[tid];
        if constexpr (PBF) {
            const uint4 pw = reinterpret_cast<const uint4*>(st.p)[tid];
            const uint32_t pp[4] = {pw.x, pw.y, pw.z, pw.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                p[2 * i] = __uint_as_float(pp[i] << 16);
                p[2 * i + 1] = __uint_as_float(pp[i] & 0xffff0000u);
            }
        } else {
            const float4 p0 = st.p[2 * tid], p1 = st.p[2 * tid + 1];
            p[0] = p0.x; p[1] = p0.y; p[2] = p0.z; p[3] = p0.w;
            p[4] = p1.x; p[5] = p1.y; p[6] = p1.z; p[7] = p1.w;
        }
        const int wm = (int)((jb_tile * G * BM) & 15) >> 2, wv = (int)((jb_tile * G * BV) & 15) >> 2;   // word offsets
        if constexpr (BM == 8) {
            const uint2 c2 = reinterpret_cast<const uint2*>(st.cm + wm)[tid];
            cm = c2.x; cm_hi = c2.y;
        } else if constexpr (BM == 2) cm = reinterpret_cast<const uint16_t*>(st.cm + wm)[tid];
        else if constexpr (BM == 4) cm = st.cm[wm + tid];
        else cm = warp_codes_finish<BM>(lane < 24 ? st.cm[wm + warp * 24 + lane] : 0u, lane);
        if constexpr (BV == 8) {
            const uint2 c2 = reinterpret_cast<const uint2*>(st.cv + wv)[tid];
            cv = c2.x; cv_hi = c2.y;
        } else if constexpr (BV == 2) cv = reinterpret_cast<const uint16_t*>(st.cv + wv)[tid];
        else if constexpr (BV == 4) cv = st.cv[wv + tid];
        else cv = warp_codes_finish<BV>(lane < 24 ? st.cv[wv + warp * 24 + lane] : 0u, lane);
        const int so = (int)(jb_tile & 3) + grp;                 // the scalars were copied from a 16-byte boundary
        dm = st.sc[0][so]; dv = st.sc[1][so]; al = st.sc[2][so];
        const uint32_t gg[4] = {gw.x, gw.y, gw.z, gw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            g[2 * i] = __uint_as_float(gg[i] << 16);
            g[2 * i + 1] = __uint_as_float(gg[i] & 0xffff0000u);
        }
    } else {
#pragma unroll
        for (int i = 0; i < EPT; ++i) {
            p[i] = 0.0f; g[i] = 0.0f;
            if (i < nv) {
                g[i] = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(gt)[tid * EPT + i] << 16);
                if constexpr (PBF)
                    p[i] = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(pt)[tid * EPT + i] << 16);
                else
                    p[i] = reinterpret_cast<const float*>(pt)[tid * EPT + i];
            }
        }
        if (have_block) {
            const uint64_t cm64 = load_codes<BM>(wcm + lane * BM), cv64 = load_codes<BV>(wcv + lane * BV);
            cm = (uint32_t)cm64; cm_hi = (uint32_t)(cm64 >> 32);
            cv = (uint32_t)cv64; cv_hi = (uint32_t)(cv64 >> 32);
            dm = __ldg(a.scale_m + jb);
            dv = __ldg(a.scale_v + jb);
            al = __ldg(a.alpha + jb);
        }
    }

    // Per-block scalars of the tile's blocks (one block per calling thread, tid < NG), from what the blocks'
    // lanes left in xin: stores the new scales and base of the blocks whose warp did not skip the tile
    // and leaves what the quantization needs in xout / xflag.
    auto block_scalars = [&]() {
        const uint4 in = s.xin[par][tid];
        const float dm_new = __uint_as_float(in.x), dv_new = __uint_as_float(in.y);
        const bool zero_m = dm_new < TINY, zero_v = dv_new < TINY;
        const float inv_dm = 1.0f / dm_new;
        const float inv_dv = 1.0f / dv_new;
        const float rho = fminf(fmaxf(__uint_as_float(in.z) * inv_dv, RHO_MIN), RHO_MAX);
        const float lam = log2_sp(rho) * (1.0f / (float)(KV - 1));
        const float al_new = fixed_base ? a.fixed_alpha : exp2_sp(lam);
        const float inv_lambda = 1.0f / log2_sp(al_new);
        const float guard = __fmaf_rn(fabsf(inv_lambda), LG2_ABS, LG2_REL * (float)(KV + 1));
        s.xout[par][tid] = make_float4(inv_dm, inv_dv, inv_lambda, 0.5f - guard);
        s.xflag[par][tid] = (zero_m ? 1u : 0u) | (zero_v ? 2u : 0u);
        const bool blk_exists = FULL || (int64_t)tid * B < rem_tile;
        if (blk_exists && in.w == 0u) {
            const int64_t j = jb_tile + tid;
            a.scale_m[j] = zero_m ? 0.0f : dm_new;
            a.scale_v[j] = zero_v ? 0.0f : dv_new;
            a.alpha[j] = zero_v ? 0.5f : al_new;
        }
    };

    // A warp in which any lane gave up waiting for its inputs leaves the tile alone: it stores nothing
    // (parameters and state keep their old values), flags its blocks for the first warp and only keeps the
    // CTA's two barriers and, if it is the first warp, the other warps' scalars going.  Blocks of 2048 span
    // the CTA, which decides as a whole and has nothing to keep going.
    if (FULL) {
        if constexpr (G == CTA) {
            if (__syncthreads_or(ah.failed ? 1 : 0)) return;
        } else if (__any_sync(0xffffffffu, ah.failed)) {
            if (gl == 0) s.xin[par][grp] = make_uint4(0u, 0u, 0u, 1u);
            bar_sync(1);
            if (tid < NG) block_scalars();
            bar_sync(2);
            return;
        }
    }

    // ---- per-block level tables: alpha^k Delta_v and y_k Delta_m (Eq. 2) ----
    // 8-bit second moments: the table holds the product of the first four factors of the
    // square-and-multiply chain (alpha^(q & 15)); the other four are multiplied on per element.
    // 8-bit first moments: no table, the codebook entry is scaled per element.
    constexpr int KVT = BV == 8 ? 16 : KV;
    float* const tab = s.tab[grp];
    float a2[BV];
    a2[0] = al;
#pragma unroll
    for (int i = 1; i < BV; ++i) a2[i] = a2[i - 1] * a2[i - 1];
    {
#pragma unroll
        for (int r0 = 0; r0 < KVT; r0 += G)
            if (r0 + gl < KVT) {
                if constexpr (BV == 8) {
                    const float a2lo[4] = {a2[0], a2[1], a2[2], a2[3]};
                    tab[r0 + gl] = pow_sm<4>(a2lo, (uint32_t)(r0 + gl));
                } else {
                    tab[r0 + gl] = pow_sm<BV>(a2, (uint32_t)(r0 + gl)) * dv;
                }
            }
        if constexpr (BM != 8) {
#pragma unroll
            for (int r0 = 0; r0 < KM; r0 += G)
                if (r0 + gl < KM) tab[KVT + r0 + gl] = s_y[r0 + gl] * dm;
        }
    }
    if constexpr (G == CTA) __syncthreads(); else __syncwarp();

    if (l2) {
#pragma unroll
        for (int i = 0; i < EPT; ++i) g[i] = __fmaf_rn(a.weight_decay, p[i], g[i]);
    }

    // ---- Eq. 2, Eq. 3, Adam(W) ----
    float mh[EPT], vh[EPT];
    uint32_t mx_v = 0;
    float mx_m_f = 0.0f;                                         // max |m^|, NaN if any is
    const char* const tab_v = reinterpret_cast<const char*>(tab);
    const char* const tab_m = reinterpret_cast<const char*>(tab + KVT);
    const CodeOffsets<BM> om4(cm, cm_hi);
    const CodeOffsets<BV> ov4(cv, cv_hi);
    // the loop is instantiated twice so that the optimizer variant costs nothing per element
    auto ema = [&](auto belief_tag) {
        constexpr bool BELIEF = decltype(belief_tag)::value;
#pragma unroll
    for (int i = 0; i < EPT; ++i) {
        float mt, vt;
        if constexpr (BM == 8) mt = *reinterpret_cast<const float*>(reinterpret_cast<const char*>(s_y) + om4(i)) * dm;
        else mt = *reinterpret_cast<const float*>(tab_m + om4(i));
        if constexpr (BV == 8) {
            float r = *reinterpret_cast<const float*>(tab_v + ov4.low4(i));
#pragma unroll
            for (int k = 4; k < 8; ++k) r = r * (ov4.bit(i, k) ? a2[k] : 1.0f);
            vt = r * dv;
        } else {
            vt = *reinterpret_cast<const float*>(tab_v + ov4(i));
        }
        const float gi = g[i];
        mh[i] = __fmaf_rn(a.beta1, mt, a.omb1 * gi);
        if (BELIEF) {                                            // AdaBelief: (g - m^)^2, plus eps
            const float sig = gi - mh[i];
            vh[i] = __fmaf_rn(a.beta2, vt, a.omb2 * (sig * sig)) + a.eps;
        } else {
            vh[i] = __fmaf_rn(a.beta2, vt, a.omb2 * (gi * gi));
        }
        const bool valid = FULL || i < nv;
        mx_m_f = max_abs_nan(mx_m_f, valid ? mh[i] : 0.0f);
        mx_v = max(mx_v, valid ? __float_as_uint(vh[i]) : 0u);
    }
    };
    if (belief) ema(std::true_type{}); else ema(std::false_type{});
    uint32_t mx_m = __float_as_uint(mx_m_f);

    // Adam(W) update of element i and, after every fourth, the store; issued between the
    // rounds of the selection below, which it does not depend on
    const Origin org = origin_of(a, tensor);
    const uint64_t ctr = org.ctr0 + (uint64_t)(uint32_t)tin * (TILE / EPT) + (uint32_t)tid;   // position in the stream: element index / 8
    uint32_t wp[4] = {0u, 0u, 0u, 0u};                          // draws of the stochastic bf16 rounding
    const bool sr = PBF && a.param_sr;
    if (PBF && !FULL && sr)
        philox_rk((uint32_t)ctr, (uint32_t)(ctr >> 32), a.step32, org.stream * 4u + 2u, a.rk, wp);
    auto update = [&](int i) {
        if constexpr (PBF) {
            const float den = __fmaf_rn(__fsqrt_rn(vh[i]), a.inv_sqrt_bc2, a.eps);
            p[i] = __fmaf_rn(-a.step_size, __fdiv_rn(mh[i], den), p[i] * a.decay);
            if (FULL) {
                if (i == 7) {
                    uint32_t pp[4];
                    if (sr) {
                        philox_rk((uint32_t)ctr, (uint32_t)(ctr >> 32), a.step32, org.stream * 4u + 2u, a.rk, wp);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            pp[j] = bf16_sr(p[2 * j], wp[j] & 0xFFFFu) | (bf16_sr(p[2 * j + 1], wp[j] >> 16) << 16);
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(p[2 * j], p[2 * j + 1]);
                            pp[j] = *reinterpret_cast<const uint32_t*>(&h);
                        }
                    }
                    __stcs(reinterpret_cast<uint4*>(pt) + tid, make_uint4(pp[0], pp[1], pp[2], pp[3]));
                }
            } else if (i < nv) {
                reinterpret_cast<uint16_t*>(pt)[tid * EPT + i] =
                    sr ? (uint16_t)bf16_sr(p[i], draw16(wp, i))
                       : __bfloat16_as_ushort(__float2bfloat16_rn(p[i]));
            }
            return;
        }
        const float den = __fmaf_rn(sqrt_approx(vh[i]), a.inv_sqrt_bc2, a.eps);
        const float rc = rcp_approx(den);
        const float q0 = mh[i] * rc;
        const float q1 = __fmaf_rn(__fmaf_rn(-den, q0, mh[i]), rc, q0);
        p[i] = __fmaf_rn(-a.step_size, q1, p[i] * a.decay);
        if (FULL) {
            if (i == 3) __stcs(reinterpret_cast<float4*>(pt) + 2 * tid, make_float4(p[0], p[1], p[2], p[3]));
            if (i == 7) __stcs(reinterpret_cast<float4*>(pt) + 2 * tid + 1, make_float4(p[4], p[5], p[6], p[7]));
        } else {
            if (i < nv) reinterpret_cast<float*>(pt)[tid * EPT + i] = p[i];
        }
    };

    // ---- block scales and the p-quantile of v^ (Sec. 3.2.2) ----
    uint32_t x_p = 0;
    if constexpr (G == CTA) {
        // one block per tile: maxima over the CTA through shared memory, radix select
        // (and the minimum of v^ over the elements that exist: the select works on the block's own range)
        uint32_t mn_v = 0xFFFFFFFFu;
        if (!fixed_base) {
#pragma unroll
            for (int i = 0; i < EPT; ++i) mn_v = min(mn_v, (FULL || i < nv) ? __float_as_uint(vh[i]) : 0xFFFFFFFFu);
            mn_v = __reduce_min_sync(0xffffffffu, mn_v);
        }
        mx_m = __reduce_max_sync(0xffffffffu, mx_m);
        mx_v = __reduce_max_sync(0xffffffffu, mx_v);
        if (lane == 0) {
            s.red[par][warp] = mx_m;
            s.red[par][8 + warp] = mx_v;
            s.red[par][16 + warp] = mn_v;
        }
#pragma unroll
        for (int i = 0; i < EPT; ++i) update(i);
        __syncthreads();
        const uint32_t t = s.red[par][lane & 15];
        mx_m = __reduce_max_sync(0xffffffffu, (lane & 8) ? 0u : t);
        mx_v = __reduce_max_sync(0xffffffffu, (lane & 8) ? t : 0u);
        if (!fixed_base) {
            uint32_t key[EPT];
#pragma unroll
            for (int i = 0; i < EPT; ++i) key[i] = (FULL || i < nv) ? __float_as_uint(vh[i]) : 0xFFFFFFFFu;
            int k = a.k_full;
            if (!FULL) {
                k = (int)ceil((double)a.p_quantile * (double)nb);
                k = min(max(k, 1), nb);
            }
            mn_v = __reduce_min_sync(0xffffffffu, s.red[par][16 + (lane & 7)]);
            x_p = cta_select(key, k, &s.sort[0][0], mn_v, mx_v);
        }
    } else {
        mx_m = seg_max31<G>(mx_m, hi);
        mx_v = seg_max31<G>(mx_v, hi);
        if (fixed_base) {                                            // no quantile to find
#pragma unroll
            for (int i = 0; i < EPT; ++i) update(i);
        } else {
            uint32_t key[EPT];
#pragma unroll
            for (int i = 0; i < EPT; ++i) key[i] = (FULL || i < nv) ? __float_as_uint(vh[i]) : KEY_MAX;
            sort8(key);
            uint32_t* const col = &s.sort[0][tid];
#pragma unroll
            for (int j = 1; j < EPT; ++j) col[(j - 1) * CTA] = key[j] ^ vflip;
            const uint32_t head = key[0] ^ vflip;
            uint32_t xv;
            if (FULL) {
                xv = select_kth<G, true>(head, col, a.k_full, hi, update);
            } else {
                int k = (int)ceil((double)a.p_quantile * (double)nb);
                k = min(max(k, 1), nb);                              // 0 for a group without a block
                xv = select_kth<G, false>(head, col, k, hi, update);
            }
            x_p = xv ^ vflip;
        }
    }

    // ---- per-block scalars, once per block, by the first warp; the others draw xi meanwhile ----
    if (gl == 0) s.xin[par][grp] = make_uint4(mx_m, mx_v, x_p, 0u);   // .w != 0: the block's warp skipped the tile
    bar_sync(1);
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    if (warp != 0) {
        if (round_v) philox_rk((uint32_t)ctr, (uint32_t)(ctr >> 32), a.step32, org.stream * 4u, a.rk, w);
    } else if (tid < NG) {
        block_scalars();
    }
    bar_sync(2);
    if (warp == 0 && round_v)
        philox_rk((uint32_t)ctr, (uint32_t)(ctr >> 32), a.step32, org.stream * 4u, a.rk, w);
    float dr[EPT];                                               // the 16-bit draws d as binary32
#pragma unroll
    for (int i = 0; i < 4; ++i) halves_to_float(w[i], dr[2 * i], dr[2 * i + 1]);
    const float4 sc = s.xout[par][grp];
    const uint32_t zf = s.xflag[par][grp];

    // ---- first moment: nearest level (Eq. 1) ----
    uint32_t om = 0, om_hi = 0;                                   // om_hi: elements 4..7 of 8-bit codes
    {
        const float inv = sc.x;
        if constexpr (BM == 2 && FULL) {
            // code = number of midpoints below r.  Each "r > mid" is evaluated on the FMA pipe as
            // the saturation of (r - mid) * 2^100: the fused multiply-add rounds the exact
            // difference, which is zero or at least 2^-30 in magnitude, so the result is exactly
            // 0 or 1 (a NaN saturates to 0, as the comparison would give).  The eight 2-bit codes
            // are accumulated in binary32 (16 bits: exact).
            constexpr float BIG = 0x1p100f;
            const float n0 = -s_mid[0] * BIG, n1 = -s_mid[1] * BIG, n2 = -s_mid[2] * BIG;
            float omf = 0.0f;
#pragma unroll
            for (int i = EPT - 1; i >= 0; --i) {
                const float r = mh[i] * inv;
                omf = __fmaf_rn(omf, 4.0f, __saturatef(__fmaf_rn(r, BIG, n0)));
                omf += __saturatef(__fmaf_rn(r, BIG, n1));
                omf += __saturatef(__fmaf_rn(r, BIG, n2));
            }
            om = (uint32_t)omf;
        } else if constexpr (BM == 3 && FULL && G != CTA) {
            // the same for all seven midpoints (measured faster than the 3-step table search, whose
            // look-ups and compares run on the busier pipes, except with blocks of 2048, where the seven
            // thresholds cost registers the CTA-wide select needs); eight 3-bit codes are 24 bits: exact in binary32
            constexpr float BIG = 0x1p100f;
            float n[7];
#pragma unroll
            for (int k = 0; k < 7; ++k) n[k] = -s_mid[k] * BIG;
            float omf = 0.0f;
#pragma unroll
            for (int i = EPT - 1; i >= 0; --i) {
                const float r = mh[i] * inv;
                omf = __fmaf_rn(omf, 8.0f, __saturatef(__fmaf_rn(r, BIG, n[0])));
#pragma unroll
                for (int k = 1; k < 7; ++k) omf += __saturatef(__fmaf_rn(r, BIG, n[k]));
            }
            om = (uint32_t)omf;
        } else if constexpr (BM == 4 && FULL) {
            // two levels of three such comparisons: mid[3], mid[7], mid[11] give the quarter s of the
            // codebook, the three midpoints inside it come from a table row addressed by s (s_mid4: the
            // midpoints times -2^100); code = 4 s + their count.  Four codes (16 bits) per accumulator.
            constexpr float BIG = 0x1p100f;
            const float nq0 = -s_mid[3] * BIG, nq1 = -s_mid[7] * BIG, nq2 = -s_mid[11] * BIG;
            float omf[2] = {0.0f, 0.0f};
#pragma unroll
            for (int i = EPT - 1; i >= 0; --i) {
                const float r = mh[i] * inv;
                const float c0 = __saturatef(__fmaf_rn(r, BIG, nq0));
                const float c1 = __saturatef(__fmaf_rn(r, BIG, nq1));
                const float c2 = __saturatef(__fmaf_rn(r, BIG, nq2));
                // 2^23 + 16 s: the low bits of the pattern are the byte offset of row s
                const float t = __fmaf_rn(c2, 16.0f, __fmaf_rn(c1, 16.0f, __fmaf_rn(c0, 16.0f, 8388608.0f)));
                const float4 row = *reinterpret_cast<const float4*>(reinterpret_cast<const char*>(s_mid4) + (__float_as_uint(t) & 0x30u));
                float code = __fmaf_rn((c0 + c1) + c2, 4.0f, __saturatef(__fmaf_rn(r, BIG, row.x)));
                code += __saturatef(__fmaf_rn(r, BIG, row.y));
                code += __saturatef(__fmaf_rn(r, BIG, row.z));
                omf[i >> 2] = __fmaf_rn(omf[i >> 2], 16.0f, code);
            }
            om = (uint32_t)omf[0] | ((uint32_t)omf[1] << 16);
        } else if constexpr (BM == 2) {
            const float mid0 = s_mid[0], mid1 = s_mid[1], mid2 = s_mid[2];
#pragma unroll
            for (int i = EPT - 1; i >= 0; --i) {
                const float r = mh[i] * inv;
                const bool c1 = r > mid1;
                const bool c0 = r > (c1 ? mid2 : mid0);
                const uint32_t q = (c1 ? 2u : 0u) + (c0 ? 1u : 0u);
                om = (om << BM) + ((FULL || i < nv) ? q : 0u);
            }
        } else {
#pragma unroll
            for (int i = EPT - 1; i >= 0; --i) {
                const float r = mh[i] * inv;
                uint32_t q = 0;
#pragma unroll
                for (int st = KM / 2; st >= 1; st >>= 1)
                    if (r > s_mid[q + st - 1]) q += st;
                uint32_t& dst = (BM == 8 && i >= 4) ? om_hi : om;
                dst = (dst << BM) + ((FULL || i < nv) ? q : 0u);
            }
        }
    }

    // ---- second moment: Eq. 6 ----
    // t = log_alpha(r) + xi is evaluated divided by K - 1, so that the clamp to [0, K-1] is the
    // saturation of the fused multiply-add; adding 1.5 * 2^23 to (K-1) * t rounds it to an integer.
    uint32_t ov = 0, ov_hi = 0;
    {
        const float inv = sc.y, il = sc.z, lim = sc.w;
        constexpr float KM1 = (float)(KV - 1);
        constexpr float MAGIC = 12582912.0f;
        constexpr uint32_t MAGIC_BITS = 0x4B400000u;
        const float ils = il * (1.0f / KM1);
        // xi = (d + 1/2) / 2^16 - 1/2 (exact); scaled copy for the approximate path
        const float xs1 = round_v ? (float)(0x1p-16 / (KV - 1)) : 0.0f;
        const float xs0 = round_v ? (float)((-0.5 + 0x1p-17) / (KV - 1)) : 0.0f;
        float worst = 0.0f;
        uint32_t acc = 0, acc_hi = 0;
#pragma unroll
        for (int i = EPT - 1; i >= 0; --i) {
            const float r = vh[i] * inv;
            const float ts = __saturatef(__fmaf_rn(lg2_approx(r), ils, __fmaf_rn(dr[i], xs1, xs0)));
            const float u = __fmaf_rn(ts, KM1, MAGIC);
            worst = fmaxf(worst, fabsf(__fmaf_rn(ts, KM1, MAGIC - u)));
            uint32_t& dst = (BV == 8 && i >= 4) ? acc_hi : acc;
            dst = dst * (1u << BV) + ((FULL || i < nv) ? __float_as_uint(u) : MAGIC_BITS);
        }
        uint32_t magic_sum = 0;
#pragma unroll
        for (int i = 0; i < (BV == 8 ? 4 : EPT); ++i) magic_sum = (magic_sum << BV) + MAGIC_BITS;
        ov = acc - magic_sum;
        if constexpr (BV == 8) ov_hi = acc_hi - magic_sum;
        if (__any_sync(0xffffffffu, worst > lim)) {
            // some element of the warp is too close to a rounding boundary for the
            // approximate logarithm: evaluate the exact sequence for all eight
            const float x1 = round_v ? 0x1p-16f : 0.0f, x0 = round_v ? -0.5f + 0x1p-17f : 0.0f;
            ov = 0;
            ov_hi = 0;
#pragma unroll
            for (int i = EPT - 1; i >= 0; --i) {
                const float r = vh[i] * inv;
                uint32_t q = KV - 1;
                if (!(r < TINY)) {
                    float t = __fmaf_rn(log2_sp(r), il, __fmaf_rn(dr[i], x1, x0));
                    t = fminf(fmaxf(t, 0.0f), KM1);
                    q = (uint32_t)__float2int_rn(t);
                }
                uint32_t& dst = (BV == 8 && i >= 4) ? ov_hi : ov;
                dst = (dst << BV) + ((FULL || i < nv) ? q : 0u);
            }
        }
    }
    if (zf & 1u) { om = 0; om_hi = 0; }
    if (zf & 2u) { ov = 0; ov_hi = 0; }

    // ---- store the codes ----
    if (FULL) {
        if constexpr (BM == 8) __stcs(reinterpret_cast<uint2*>(wcm) + lane, make_uint2(om, om_hi));
        else warp_store_codes<BM>(wcm, lane, om);
        if constexpr (BV == 8) __stcs(reinterpret_cast<uint2*>(wcv) + lane, make_uint2(ov, ov_hi));
        else warp_store_codes<BV>(wcv, lane, ov);
    } else if (have_block) {
        store_codes<BM>(wcm + lane * BM, ((uint64_t)om_hi << 32) | om);
        store_codes<BV>(wcv + lane * BV, ((uint64_t)ov_hi << 32) | ov);
    }
}

template <int BM, int BV, int G, bool PBF, bool PLAIN>
__global__ void __launch_bounds__(CTA, (BM == 8 || BV == 8) ? 3 : 4) solo_step_fast_kernel(const StepArgs a) {
    constexpr int KM = 1 << BM;
    extern __shared__ __align__(16) unsigned char fast_smem[];   // sizeof(FastShared<BM, BV>), above the static 48 KB limit
    FastShared<BM, BV>& s = *reinterpret_cast<FastShared<BM, BV>*>(fast_smem);
    __shared__ float s_y[KM];
    __shared__ float s_mid[KM];
    __shared__ float4 s_mid4[4];     // 4-bit first moments: per quarter of the codebook, its three inner midpoints times -2^100
    const int tid = threadIdx.x;
    for (int i = tid; i < KM; i += CTA) {
        s_y[i] = a.tables[i];
        if (i < KM - 1) s_mid[i] = a.tables[KM + i];
    }
    if (BM == 4 && tid < 4)
        s_mid4[tid] = make_float4(-a.tables[KM + 4 * tid] * 0x1p100f, -a.tables[KM + 4 * tid + 1] * 0x1p100f,
                                  -a.tables[KM + 4 * tid + 2] * 0x1p100f, 0.0f);
    for (int r = 7; r < 16; ++r) s.sort[r][tid] = (G == 16 && (tid & G)) ? ~KEY_MAX : KEY_MAX;   // sentinels, v domain
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s.mbar[0])) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s.mbar[1])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // Tile indices fit 32 bits (the host selects this kernel only below 2^31 - 2^20 tiles).  With
    // sub-CTA blocks a CTA takes a contiguous share of the launch's tiles, so that its next tile is
    // nearly always the next tile of the same tensor and can be copied ahead even in sets of small
    // tensors (with tiles dealt out in turn it rarely was; measured +7 % on the GPT-125M set, +16 %
    // on the ragged set, +2 % on the 7B set).  Blocks of 2048 measured 7 % slower that way and keep
    // tiles dealt in turn.  Tiles are visited in increasing order, so the tensor of a tile is found by
    // a search for the CTA's first tile and by walking forward after that.
    const int launch_tiles = (int)(a.total_tiles - a.tile_first);
    const int share = (launch_tiles + (int)gridDim.x - 1) / (int)gridDim.x;
    const int step = G == CTA ? (int)gridDim.x : 1;            // to the CTA's next tile
    const int tile_begin = (int)min(a.tile_first + (int64_t)blockIdx.x * (G == CTA ? 1 : share), a.total_tiles);
    const int tile_end = G == CTA ? (int)a.total_tiles : (int)min((int64_t)tile_begin + share, a.total_tiles);
    int tensor = (a.num_tensors > 1 && tile_begin < tile_end ? find_tensor(a.tile_start, a.num_tensors, tile_begin) : 0) - 1;
    int t_lo = 0, t_hi = 0, full_tiles = 0;      // the tensor's tiles [t_lo, t_hi); its first full_tiles are full
    int64_t jb0 = 0;
    char* pbase = nullptr;
    const char* gbase = nullptr;
    bool skip = false;
    Ahead ah;
    int par = 0;
    for (int tile = tile_begin; tile < tile_end; tile += step) {
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
            skip = a.numel_check != nullptr && __ldg(a.numel_check + tensor) != n;
            if (skip && tid == 0) atomicOr(a.status, 1);
        }
        if (skip) continue;
        const int tin = tile - t_lo;
        if (a.only_partial && tin < full_tiles) {                 // another launch did the full tiles
            if (step == 1) tile = t_lo + full_tiles - 1;          // on to the tensor's first tile that is not full
            continue;
        }
        const int64_t jb_tile = jb0 + (int64_t)tin * (CTA / G);
        if (tin < full_tiles)
            fast_tile<BM, BV, G, true, PBF, PLAIN>(a, s, s_y, s_mid, s_mid4, pbase, gbase, 0, tin, jb_tile, tensor, par, ah,
                                       tin + step < full_tiles && tile + step < tile_end, step, tile);
        else
            fast_tile<BM, BV, G, false, PBF, PLAIN>(a, s, s_y, s_mid, s_mid4, pbase, gbase, __ldg(a.numel + tensor), tin, jb_tile,
                                                    tensor, par, ah, false, 0, tile);
        par ^= 1;
    }
    // A thread that gave up on a copy waits once more, again bounded, for the last one that was issued,
    // so that no copy is still writing to a stage when the CTA's shared memory is released.
    if (ah.failed && ah.fill > 0) {
        const uint32_t last = ah.fill - 1u;
        mbar_wait(smem_u32(&s.mbar[last & 1u]), (last >> 1) & 1u);
    }
}

}  // namespace solo
