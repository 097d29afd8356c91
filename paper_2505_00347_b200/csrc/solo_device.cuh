// Device code of the fused SOLO optimizer step for sm_100a.
//
// One kernel does the whole step for a tile of TILE elements of one tensor:
// load -> dequantize (Eq. 2) -> EMA (Eq. 3) -> Adam(W) update -> block scales ->
// p-quantile and base of the logarithmic codebook -> quantize (Eq. 1/5/6) -> pack
// -> store.  Every thread owns EPT = 8 consecutive elements; a quantization block
// of B elements is owned by G = B/8 consecutive threads (a sub-warp group for
// B <= 256, the whole CTA for B = 2048).
//
// Arithmetic is IEEE binary32, round to nearest, with fused multiply-adds only
// where written (compile with -fmad=false); log2 / exp2 are fixed polynomial
// sequences so that the rounded logarithm of Eq. 6 is reproducible bit for bit.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace solo {

constexpr int EPT = 8;                 // elements per thread
constexpr int CTA = 256;               // threads per CTA
constexpr int TILE = EPT * CTA;        // elements per tile (2048)

constexpr float TINY = 0x1p-100f;      // scales below this are stored as zero
constexpr float RHO_MIN = 0x1p-48f;    // clamp of x_p / Delta
constexpr float RHO_MAX = 1.0f - 0x1p-10f;

struct StepArgs {
    // tensors: either device arrays of pointers (multi) or the two direct pointers
    void* const* param_list;
    const void* const* grad_list;
    const int64_t* numel_check;        // caller's numel array (device) or null
    void* param_single;
    const void* grad_single;
    // geometry (device arrays owned by the state)
    const int64_t* numel;              // [T]
    const int64_t* block_start;        // [T+1]
    const int64_t* tile_start;         // [T+1]
    int32_t num_tensors;
    int64_t total_tiles;               // the launch covers tiles [tile_first, total_tiles)
    int64_t tile_first;
    int32_t only_partial;              // streamlined and general kernel: skip full tiles of aligned tensors (another launch did them)
    int64_t debug_stall_tile_p1;       // test hook of the staged kernels: 1 + the number of the tile whose input copy
                                       // announces 16 bytes more than it brings (the wait for it runs out); 0: none
    // state
    uint8_t* codes_m;
    uint8_t* codes_v;
    float* scale_m;
    float* scale_v;
    float* alpha;
    const float* tables;               // y[K], mid[K-1], inv_gap[K-1] of the first-moment codebook
    const float* tables_v;             // baseline second-moment codebook y[K], mid[K-1]; null: Eq. 6
    int* status;                       // device word: non-zero after a descriptor mismatch
    // Position of every tensor of the list in the random stream (device arrays, never null; all zeros:
    // "tensor t of the list is stream t, from its first element"): a shard of a larger tensor names the
    // tensor's stream and the stream position (element index / 8) of the shard's first element.
    const int32_t* origin_id;          // [T] stream number minus the tensor's position in the list
    const int64_t* origin_ctr;         // [T]
    // hyper-parameters, already reduced to what the kernel multiplies with
    float beta1, beta2, omb1, omb2, step_size, inv_sqrt_bc2, eps, decay, weight_decay, p_quantile;
    float fixed_alpha;                 // in (0,1): base of every block; 0: base from the p-quantile
    int32_t l2, round_m, round_v, param_bf16, block, k_full, belief;
    int32_t param_sr;                  // bf16 parameters are rounded stochastically (Philox purpose 2)
    uint32_t seed_lo, seed_hi, step32;
    // Philox round keys (seed + r * Weyl constant), r = 0..9: [2r] low word, [2r+1] high word
    uint32_t rk[20];
};

// ---------------------------------------------------------------------------
// log2 / exp2 as fixed IEEE operation sequences (see the block comment above).
// ---------------------------------------------------------------------------
__device__ __forceinline__ float log2_sp(float x) {
    // x = 2^e * m, m in [sqrt(1/2), sqrt(2)); log2(m) = f * P(f), f = m - 1
    int i = __float_as_int(x);
    int e = (i - 0x3F3504F3) >> 23;
    float m = __int_as_float(i - (e << 23));
    float f = m - 1.0f;
    float p = 0x1.01b6dep-3f;
    p = __fmaf_rn(p, f, -0x1.a87d0ep-3f);
    p = __fmaf_rn(p, f, 0x1.b9c91ap-3f);
    p = __fmaf_rn(p, f, -0x1.e95be6p-3f);
    p = __fmaf_rn(p, f, 0x1.26d384p-2f);
    p = __fmaf_rn(p, f, -0x1.715c4ep-2f);
    p = __fmaf_rn(p, f, 0x1.ec73d6p-2f);
    p = __fmaf_rn(p, f, -0x1.71547p-1f);
    p = __fmaf_rn(p, f, 0x1.715476p+0f);
    return __fmaf_rn(f, p, (float)e);
}

__device__ __forceinline__ float exp2_sp(float x) {
    // n = rint(x), 2^(x-n) by a degree-6 polynomial, exponent advanced by n
    float n = rintf(x);
    float f = x - n;
    float p = 0x1.41d33cp-13f;
    p = __fmaf_rn(p, f, 0x1.5f456ap-10f);
    p = __fmaf_rn(p, f, 0x1.3b2dbcp-7f);
    p = __fmaf_rn(p, f, 0x1.c6aed4p-5f);
    p = __fmaf_rn(p, f, 0x1.ebfbdap-3f);
    p = __fmaf_rn(p, f, 0x1.62e43p-1f);
    p = __fmaf_rn(p, f, 1.0f);
    return __int_as_float(__float_as_int(p) + ((int)n << 23));
}

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11).
// ---------------------------------------------------------------------------
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The Philox stream of tensor `tensor` of the list and the counter of its first element.
struct Origin {
    uint32_t stream;
    uint64_t ctr0;
};
__device__ __forceinline__ Origin origin_of(const StepArgs& a, int tensor) {
    Origin o;
    o.stream = (uint32_t)(tensor + __ldg(a.origin_id + tensor));
    o.ctr0 = (uint64_t)__ldg(a.origin_ctr + tensor);
    return o;
}

// 16-bit draw of element i (0..7) of a thread's eight: halfword i of the Philox block.
// binary32 -> bf16 bit pattern with a 16-bit draw: the upper neighbour is taken with
// probability (dropped bits) / 2^16; infinities and NaN are truncated (NaN kept quiet).
__device__ __forceinline__ uint32_t bf16_sr(float x, uint32_t d) {
    const uint32_t u = __float_as_uint(x);
    if ((u & 0x7F800000u) == 0x7F800000u) return (u >> 16) | ((u & 0x007FFFFFu) ? 0x0040u : 0u);
    return (u + d) >> 16;
}

__device__ __forceinline__ uint32_t draw16(const uint32_t (&w)[4], int i) {
    return (i & 1) ? (w[i >> 1] >> 16) : (w[i >> 1] & 0xFFFFu);
}

// ---------------------------------------------------------------------------
// Group collectives.  G <= 32: `mask` names the group's lanes.  G = 256: the
// whole CTA cooperates through shared memory.
// ---------------------------------------------------------------------------
template <bool CTA_GROUP>
__device__ __forceinline__ uint32_t group_max(uint32_t v, uint32_t mask, uint32_t* s_red) {
    if constexpr (!CTA_GROUP) {
        return __reduce_max_sync(mask, v);
    } else {
        v = __reduce_max_sync(0xffffffffu, v);
        __syncthreads();                       // s_red may still be read from the last use
        if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
        __syncthreads();
        uint32_t w = s_red[threadIdx.x & 7];
        return __reduce_max_sync(0xffffffffu, w);
    }
}

__device__ __forceinline__ void cswap(uint32_t& a, uint32_t& b) {
    uint32_t lo = min(a, b), hi = max(a, b);
    a = lo; b = hi;
}

// k-th smallest (1-based) of the group's keys; exact, ties included.
// Sub-warp groups: every lane sorts its 8 keys, then the group pops its minimum
// until k keys have been counted.  s_sort is [EPT][CTA] words.
template <bool CTA_GROUP>
__device__ __forceinline__ uint32_t group_select(uint32_t (&key)[EPT], int k, uint32_t mask,
                                                 uint32_t* s_sort, uint32_t* s_hist) {
    if constexpr (!CTA_GROUP) {
        cswap(key[0], key[1]); cswap(key[2], key[3]); cswap(key[4], key[5]); cswap(key[6], key[7]);
        cswap(key[0], key[2]); cswap(key[1], key[3]); cswap(key[4], key[6]); cswap(key[5], key[7]);
        cswap(key[1], key[2]); cswap(key[5], key[6]); cswap(key[0], key[4]); cswap(key[3], key[7]);
        cswap(key[1], key[5]); cswap(key[2], key[6]);
        cswap(key[1], key[4]); cswap(key[3], key[6]);
        cswap(key[2], key[4]); cswap(key[3], key[5]);
        cswap(key[3], key[4]);
        // Row j of the lane's column holds its (j+1)-th smallest key; row 0 holds the
        // "exhausted" sentinel, so that popping is one unconditional load and two selects
        // (no divergent branch between the warp-synchronous operations of the loop).
        uint32_t* mine = s_sort + threadIdx.x;
        mine[0] = 0xFFFFFFFFu;
#pragma unroll
        for (int j = 1; j < EPT; ++j) mine[j * CTA] = key[j];
        uint32_t head = key[0];
        int ptr = 0, cnt = 0;
        uint32_t gmin;
        while (true) {
            gmin = __reduce_min_sync(mask, head);
            const bool eq = head == gmin;
            cnt += __popc(__ballot_sync(mask, eq));
            if (cnt >= k) break;
            const int np = ptr + 1;
            const uint32_t nxt = mine[(np & (EPT - 1)) * CTA];
            head = eq ? nxt : head;
            ptr = eq ? np : ptr;
        }
        return gmin;
    } else {
        // radix select, 8 bits per pass, 256 threads = 256 bins
        uint32_t prefix = 0;
        int kk = k;
        const int tid = threadIdx.x;
        uint32_t* s_scan = s_hist + 256;       // [8] warp totals, [8] = chosen bin, [9] = new rank
#pragma unroll 1
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            __syncthreads();
            s_hist[tid] = 0;
            __syncthreads();
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                bool in = pass == 0 || (key[i] >> (shift + 8)) == prefix;
                if (in) atomicAdd(&s_hist[(key[i] >> shift) & 255u], 1u);
            }
            __syncthreads();
            uint32_t c = s_hist[tid], incl = c;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                uint32_t t = __shfl_up_sync(0xffffffffu, incl, d);
                if ((tid & 31) >= d) incl += t;
            }
            if ((tid & 31) == 31) s_scan[tid >> 5] = incl;
            __syncthreads();
            uint32_t base = 0;
#pragma unroll
            for (int w = 0; w < 8; ++w)
                if (w < (tid >> 5)) base += s_scan[w];
            incl += base;
            uint32_t excl = incl - c;
            if ((uint32_t)kk > excl && (uint32_t)kk <= incl) {
                s_scan[8] = tid;
                s_scan[9] = kk - excl;
            }
            __syncthreads();
            prefix = (prefix << 8) | s_scan[8];
            kk = (int)s_scan[9];
        }
        return prefix;
    }
}

// ---------------------------------------------------------------------------
// Packed codes of one thread: EPT codes of `BITS` bits = BITS bytes.
// ---------------------------------------------------------------------------
template <int BITS>
__device__ __forceinline__ uint64_t load_codes(const uint8_t* p) {
    if constexpr (BITS == 2) return *reinterpret_cast<const uint16_t*>(p);
    else if constexpr (BITS == 4) return *reinterpret_cast<const uint32_t*>(p);
    else if constexpr (BITS == 8) return *reinterpret_cast<const uint64_t*>(p);
    else return (uint64_t)p[0] | ((uint64_t)p[1] << 8) | ((uint64_t)p[2] << 16);
}
template <int BITS>
__device__ __forceinline__ void store_codes(uint8_t* p, uint64_t w) {
    if constexpr (BITS == 2) *reinterpret_cast<uint16_t*>(p) = (uint16_t)w;
    else if constexpr (BITS == 4) *reinterpret_cast<uint32_t*>(p) = (uint32_t)w;
    else if constexpr (BITS == 8) *reinterpret_cast<uint64_t*>(p) = w;
    else { p[0] = (uint8_t)w; p[1] = (uint8_t)(w >> 8); p[2] = (uint8_t)(w >> 16); }
}

// alpha^q, least significant bit of q first (the multiplications by 1 are exact)
template <int BITS>
__device__ __forceinline__ float pow_sm(const float (&a2)[BITS], uint32_t q) {
    float r = (q & 1u) ? a2[0] : 1.0f;
#pragma unroll
    for (int i = 1; i < BITS; ++i) r = r * ((q >> i) & 1u ? a2[i] : 1.0f);
    return r;
}

// Tile -> tensor: largest t with tile_start[t] <= x.
__device__ __forceinline__ int find_tensor(const int64_t* __restrict__ start, int n, int64_t x) {
    int lo = 0, hi = n;                        // start[lo] <= x < start[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (__ldg(start + mid) <= x) lo = mid; else hi = mid;
    }
    return lo;
}

// ---------------------------------------------------------------------------
// The fused step.
// ---------------------------------------------------------------------------
template <int BM, int BV, bool CTA_GROUP>
__global__ void __launch_bounds__(CTA) solo_step_kernel(const StepArgs a) {
    constexpr int KM = 1 << BM, KV = 1 << BV;
    __shared__ float s_y[KM];
    __shared__ float s_mid[KM];
    __shared__ float s_gap[KM];
    __shared__ float s_yv[KV];
    __shared__ float s_midv[KV];
    __shared__ uint32_t s_sort[CTA_GROUP ? 1 : EPT * CTA];
    __shared__ uint32_t s_hist[CTA_GROUP ? 256 + 16 : 1];
    __shared__ uint32_t s_red[8];

    const int tid = threadIdx.x;
    for (int i = tid; i < KM; i += CTA) {
        s_y[i] = a.tables[i];
        if (i < KM - 1) {
            s_mid[i] = a.tables[KM + i];
            s_gap[i] = a.tables[2 * KM - 1 + i];
        }
    }
    const bool vtab = a.tables_v != nullptr;                  // baseline codebook for the second moment
    if (vtab)
        for (int i = tid; i < KV; i += CTA) {
            s_yv[i] = a.tables_v[i];
            if (i < KV - 1) s_midv[i] = a.tables_v[KV + i];
        }
    __syncthreads();

    const int B = CTA_GROUP ? TILE : a.block;
    const int G = B / EPT;                                     // threads per block
    const int lane = tid & 31;
    const uint32_t mask = CTA_GROUP || G >= 32 ? 0xffffffffu : ((1u << G) - 1u) << (lane & ~(G - 1));
    const int gl = tid & (G - 1);                              // thread within its block
    const bool bf16p = a.param_bf16 != 0;

    // Tiles are dealt out in turn.  After a launch that did the full tiles of the aligned tensors
    // (only_partial) a CTA takes a contiguous share instead and jumps over each tensor's full tiles, so
    // that it visits a few tiles per tensor of its share rather than every tile of the launch.
    const int64_t share = (a.total_tiles - a.tile_first + gridDim.x - 1) / gridDim.x;
    const int64_t tile_begin = a.only_partial ? min(a.tile_first + (int64_t)blockIdx.x * share, a.total_tiles)
                                              : a.tile_first + blockIdx.x;
    const int64_t tile_end = a.only_partial ? min(tile_begin + share, a.total_tiles) : a.total_tiles;
    const int64_t stride = a.only_partial ? 1 : (int64_t)gridDim.x;
    for (int64_t tile = tile_begin; tile < tile_end; tile += stride) {
        const int tensor = a.num_tensors > 1 ? find_tensor(a.tile_start, a.num_tensors, tile) : 0;
        const int64_t n = __ldg(a.numel + tensor);
        if (a.numel_check != nullptr && __ldg(a.numel_check + tensor) != n) {
            if (tid == 0) atomicOr(a.status, 1);
            continue;
        }
        const int64_t tin = tile - __ldg(a.tile_start + tensor);
        char* pbase = (char*)(a.param_list ? a.param_list[tensor] : a.param_single);
        const char* gbase = (const char*)(a.grad_list ? a.grad_list[tensor] : a.grad_single);
        const bool aligned = ((((uintptr_t)pbase) | ((uintptr_t)gbase)) & 15u) == 0;
        if (a.only_partial && aligned && tin < n / TILE) {           // another launch did the full tiles:
            tile += n / TILE - tin - 1;                               // on to the tensor's first tile that is not full
            continue;
        }
        const int64_t e0 = tin * TILE + (int64_t)tid * EPT;
        const int64_t blk_in_tensor = e0 / B;
        const int64_t blk_elem0 = blk_in_tensor * B;
        if (!CTA_GROUP && blk_elem0 >= n) continue;            // the whole group has no block
        const int nb = (int)min((int64_t)B, n - blk_elem0);    // valid elements of the block
        const int nv = (int)max((int64_t)0, min((int64_t)EPT, n - e0));
        const int64_t jb = __ldg(a.block_start + tensor) + blk_in_tensor;

        const bool vec = nv == EPT && aligned;

        // ---- load ----
        float p[EPT], g[EPT];
        if (vec) {
            uint4 gw = *reinterpret_cast<const uint4*>(gbase + e0 * 2);
            uint32_t gg[4] = {gw.x, gw.y, gw.z, gw.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                g[2 * i] = __uint_as_float(gg[i] << 16);
                g[2 * i + 1] = __uint_as_float(gg[i] & 0xffff0000u);
            }
            if (bf16p) {
                uint4 pw = *reinterpret_cast<const uint4*>(pbase + e0 * 2);
                uint32_t pp[4] = {pw.x, pw.y, pw.z, pw.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    p[2 * i] = __uint_as_float(pp[i] << 16);
                    p[2 * i + 1] = __uint_as_float(pp[i] & 0xffff0000u);
                }
            } else {
                float4 p0 = *reinterpret_cast<const float4*>(pbase + e0 * 4);
                float4 p1 = *reinterpret_cast<const float4*>(pbase + e0 * 4 + 16);
                p[0] = p0.x; p[1] = p0.y; p[2] = p0.z; p[3] = p0.w;
                p[4] = p1.x; p[5] = p1.y; p[6] = p1.z; p[7] = p1.w;
            }
        } else {
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                p[i] = 0.0f; g[i] = 0.0f;
                if (i < nv) {
                    g[i] = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(gbase)[e0 + i] << 16);
                    p[i] = bf16p ? __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(pbase)[e0 + i] << 16)
                                 : reinterpret_cast<const float*>(pbase)[e0 + i];
                }
            }
        }
        const int64_t slot = jb * (int64_t)(B / EPT) + gl;     // this thread's 8-element slot
        uint64_t cm = load_codes<BM>(a.codes_m + slot * BM);
        uint64_t cv = load_codes<BV>(a.codes_v + slot * BV);
        const float dm = a.scale_m[jb], dv = a.scale_v[jb], al = a.alpha[jb];

        // ---- Eq. 2, Eq. 3, Adam(W) ----
        float a2[BV];
        a2[0] = al;
#pragma unroll
        for (int i = 1; i < BV; ++i) a2[i] = a2[i - 1] * a2[i - 1];
        float mh[EPT], vh[EPT];
#pragma unroll
        for (int i = 0; i < EPT; ++i) {
            float gi = g[i];
            if (a.l2) gi = __fmaf_rn(a.weight_decay, p[i], gi);
            uint32_t qm = (uint32_t)(cm >> (i * BM)) & (KM - 1);
            uint32_t qv = (uint32_t)(cv >> (i * BV)) & (KV - 1);
            float mt = s_y[qm] * dm;
            float vt = (vtab ? s_yv[qv] : pow_sm<BV>(a2, qv)) * dv;
            mh[i] = __fmaf_rn(a.beta1, mt, a.omb1 * gi);
            const float sig = a.belief ? gi - mh[i] : gi;            // AdaBelief: (g - m^)^2, plus eps
            vh[i] = __fmaf_rn(a.beta2, vt, a.omb2 * (sig * sig));
            if (a.belief) vh[i] = vh[i] + a.eps;
            float den = __fmaf_rn(sqrtf(vh[i]), a.inv_sqrt_bc2, a.eps);
            p[i] = __fmaf_rn(-a.step_size, mh[i] / den, p[i] * a.decay);
        }

        // ---- store parameters ----
        const bool sr = bf16p && a.param_sr;
        uint32_t wp[4] = {0u, 0u, 0u, 0u};
        const Origin org = origin_of(a, tensor);
        if (sr) {
            const uint64_t c = org.ctr0 + ((uint64_t)e0 >> 3);
            philox4x32_10((uint32_t)c, (uint32_t)(c >> 32), a.step32, org.stream * 4u + 2u,
                          a.seed_lo, a.seed_hi, wp);
        }
        if (vec) {
            if (bf16p) {
                uint32_t pp[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (sr) {
                        pp[i] = bf16_sr(p[2 * i], wp[i] & 0xFFFFu) | (bf16_sr(p[2 * i + 1], wp[i] >> 16) << 16);
                    } else {
                        __nv_bfloat162 h = __floats2bfloat162_rn(p[2 * i], p[2 * i + 1]);
                        pp[i] = *reinterpret_cast<uint32_t*>(&h);
                    }
                }
                *reinterpret_cast<uint4*>(pbase + e0 * 2) = make_uint4(pp[0], pp[1], pp[2], pp[3]);
            } else {
                *reinterpret_cast<float4*>(pbase + e0 * 4) = make_float4(p[0], p[1], p[2], p[3]);
                *reinterpret_cast<float4*>(pbase + e0 * 4 + 16) = make_float4(p[4], p[5], p[6], p[7]);
            }
        } else {
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                if (i < nv) {
                    if (sr) reinterpret_cast<uint16_t*>(pbase)[e0 + i] = (uint16_t)bf16_sr(p[i], draw16(wp, i));
                    else if (bf16p) reinterpret_cast<__nv_bfloat16*>(pbase)[e0 + i] = __float2bfloat16_rn(p[i]);
                    else reinterpret_cast<float*>(pbase)[e0 + i] = p[i];
                }
            }
        }

        // ---- block scales: Delta_m = max |m^|, Delta_v = max v^ (bit patterns order like values) ----
        uint32_t mx_m = 0, mx_v = 0, key[EPT];
#pragma unroll
        for (int i = 0; i < EPT; ++i) {
            const bool valid = i < nv;
            uint32_t um = __float_as_uint(mh[i]) & 0x7fffffffu, uv = __float_as_uint(vh[i]);
            mx_m = max(mx_m, valid ? um : 0u);
            mx_v = max(mx_v, valid ? uv : 0u);
            key[i] = valid ? uv : 0xFFFFFFFFu;
        }
        mx_m = group_max<CTA_GROUP>(mx_m, mask, s_red);
        mx_v = group_max<CTA_GROUP>(mx_v, mask, s_red);
        const float dm_new = __uint_as_float(mx_m), dv_new = __uint_as_float(mx_v);
        const bool zero_m = dm_new < TINY, zero_v = dv_new < TINY;

        // ---- first moment: Eq. 1 (nearest) or Eq. 5 (stochastic) ----
        uint64_t om = 0;
        if (!zero_m) {
            const float inv = 1.0f / dm_new;
            uint32_t wm[4];
            if (a.round_m) {
                const uint64_t c = org.ctr0 + ((uint64_t)e0 >> 3);   // one Philox block per 8 elements
                philox4x32_10((uint32_t)c, (uint32_t)(c >> 32), a.step32, org.stream * 4u + 1u,
                              a.seed_lo, a.seed_hi, wm);
            }
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                const float r = mh[i] * inv;
                uint32_t q = 0;
                if (a.round_m) {
#pragma unroll
                    for (int s = KM / 2; s >= 1; s >>= 1) {
                        uint32_t c = q + s;
                        if (c <= KM - 2 && r >= s_y[c]) q = c;
                    }
                    const float frac = (r - s_y[q]) * s_gap[q];
                    const float u = (float)draw16(wm, i) * 0x1p-16f;
                    q += u < frac ? 1u : 0u;
                } else {
#pragma unroll
                    for (int s = KM / 2; s >= 1; s >>= 1)
                        if (r > s_mid[q + s - 1]) q += s;
                }
                if (i < nv) om |= (uint64_t)q << (i * BM);
            }
        }

        // ---- second moment: p-quantile, base, Eq. 6 ----
        uint64_t ov = 0;
        float al_new = 0.5f;
        if (!zero_v && vtab) {                                   // uniform: Eq. 1 on a fixed codebook
            const float inv = 1.0f / dv_new;
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                const float r = vh[i] * inv;
                uint32_t q = 0;
#pragma unroll
                for (int s = KV / 2; s >= 1; s >>= 1)
                    if (r > s_midv[q + s - 1]) q += s;
                if (i < nv) ov |= (uint64_t)q << (i * BV);
            }
        } else if (!zero_v) {                                    // uniform over the group
            int k = a.k_full;
            if (nb != B) {
                k = (int)ceil((double)a.p_quantile * (double)nb);
                k = min(max(k, 1), nb);
            }
            const float inv = 1.0f / dv_new;
            if (a.fixed_alpha > 0.0f) {                          // uniform: fixed base, no quantile
                al_new = a.fixed_alpha;
            } else {
                const float x_p = __uint_as_float(group_select<CTA_GROUP>(key, k, mask, s_sort, s_hist));
                float rho = fminf(fmaxf(x_p * inv, RHO_MIN), RHO_MAX);
                const float lam = log2_sp(rho) * (1.0f / (float)(KV - 1));
                al_new = exp2_sp(lam);
            }
            const float inv_lambda = 1.0f / log2_sp(al_new);
            uint32_t wv[4];
            if (a.round_v) {
                const uint64_t c = org.ctr0 + ((uint64_t)e0 >> 3);
                philox4x32_10((uint32_t)c, (uint32_t)(c >> 32), a.step32, org.stream * 4u,
                              a.seed_lo, a.seed_hi, wv);
            }
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                const float r = vh[i] * inv;
                const float xi = a.round_v ? (float)draw16(wv, i) * 0x1p-16f - 0.5f + 0x1p-17f : 0.0f;
                uint32_t q = KV - 1;
                if (!(r < TINY)) {
                    float t = __fmaf_rn(log2_sp(r), inv_lambda, xi);
                    t = fminf(fmaxf(t, 0.0f), (float)(KV - 1));
                    q = (uint32_t)__float2int_rn(t);
                }
                if (i < nv) ov |= (uint64_t)q << (i * BV);
            }
        }

        // ---- store the state ----
        store_codes<BM>(a.codes_m + slot * BM, om);
        store_codes<BV>(a.codes_v + slot * BV, ov);
        if (gl == 0) {
            a.scale_m[jb] = zero_m ? 0.0f : dm_new;
            a.scale_v[jb] = zero_v ? 0.0f : dv_new;
            a.alpha[jb] = al_new;
        }
    }
}

// ---------------------------------------------------------------------------
// Eq. 2 for inspection: out[elem_start[t] + e] = dequantized moment.
// ---------------------------------------------------------------------------
struct DequantArgs {
    const int64_t* numel;
    const int64_t* block_start;
    const int64_t* tile_start;
    const int64_t* elem_start;
    int32_t num_tensors;
    int64_t total_tiles;
    const uint8_t* codes;
    const float* scale;
    const float* alpha;
    const float* tables;               // y[K] of the codebook when which == 0
    float* out;
    int32_t block, which;              // which: 0 level table times scale, 1 alpha^q times scale
};

template <int BITS>
__global__ void __launch_bounds__(CTA) solo_dequant_kernel(const DequantArgs a) {
    constexpr int K = 1 << BITS;
    __shared__ float s_y[K];
    const int tid = threadIdx.x;
    if (a.which == 0)
        for (int i = tid; i < K; i += CTA) s_y[i] = a.tables[i];
    __syncthreads();
    const int B = a.block;
    for (int64_t tile = blockIdx.x; tile < a.total_tiles; tile += gridDim.x) {
        const int tensor = a.num_tensors > 1 ? find_tensor(a.tile_start, a.num_tensors, tile) : 0;
        const int64_t n = a.numel[tensor];
        const int64_t e0 = (tile - a.tile_start[tensor]) * TILE + (int64_t)tid * EPT;
        if (e0 >= n) continue;
        const int nv = (int)min((int64_t)EPT, n - e0);
        const int64_t blk = e0 / B;
        const int64_t jb = a.block_start[tensor] + blk;
        const int64_t slot = jb * (int64_t)(B / EPT) + (e0 - blk * B) / EPT;
        const uint64_t c = load_codes<BITS>(a.codes + slot * BITS);
        const float d = a.scale[jb];
        float a2[BITS];
        a2[0] = a.alpha[jb];
#pragma unroll
        for (int i = 1; i < BITS; ++i) a2[i] = a2[i - 1] * a2[i - 1];
        float* o = a.out + a.elem_start[tensor] + e0;
#pragma unroll
        for (int i = 0; i < EPT; ++i) {
            uint32_t q = (uint32_t)(c >> (i * BITS)) & (K - 1);
            float v = a.which == 0 ? s_y[q] * d : pow_sm<BITS>(a2, q) * d;
            if (i < nv) o[i] = v;
        }
    }
}

}  // namespace solo
