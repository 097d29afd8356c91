// Host side of the C ABI declared in include/solo.h: state management, argument
// validation, hyper-parameter reduction and kernel dispatch.
#include "solo.h"

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "solo_device.cuh"
#include "solo_dispatch.h"

using solo::StepArgs;

struct solo_state {
    int device = 0;
    int bits_m = 0, bits_v = 0, block = 0, num_tensors = 0;
    int64_t numel_total = 0, nblk_total = 0, tiles_total = 0;
    std::vector<int64_t> numel, block_start, tile_start, elem_start;  // host copies
    // device
    uint8_t* codes_m = nullptr;
    uint8_t* codes_v = nullptr;
    float* scale_m = nullptr;
    float* scale_v = nullptr;
    float* alpha = nullptr;
    int64_t* geom = nullptr;      // numel[T] | block_start[T+1] | tile_start[T+1] | elem_start[T+1]
    float* tables_m = nullptr;    // first-moment codebook tables for bits_m
    float* tables_v = nullptr;    // the three baseline second-moment codebooks for bits_v, each y[K] | mid[K-1]
    int v_codebook = SOLO_V_LOG;  // selector of the last step (what solo_dequant decodes with)
    int* status = nullptr;
    int32_t* origin_id = nullptr;   // [T] device: Philox stream of every tensor minus its position in the list (solo_state_set_origin)
    int64_t* origin_ctr = nullptr;  // [T] device: stream position (element index / 8) of every tensor's first element
    size_t bytes_codes_m = 0, bytes_codes_v = 0;
    struct HostPipe* pipe = nullptr;   // staging of solo_multi_step_host, created at its first call
};

// Staging of the host-buffer entry point: three slots, each with its own stream, a device buffer
// for one chunk of gradients and the device array of per-tensor gradient pointers of that chunk.
struct HostPipe {
    static constexpr int SLOTS = 3;
    int64_t chunk_tiles = 0;
    cudaStream_t stream[SLOTS] = {};
    cudaEvent_t done[SLOTS] = {};          // end of the slot's last chunk
    cudaEvent_t start = nullptr;           // the caller's stream at the call
    unsigned char* d_grad[SLOTS] = {};     // chunk_tiles * (TILE * 2 + 16) bytes
    void** d_grad_list[SLOTS] = {};        // [T] device
    void** h_grad_list[SLOTS] = {};        // [T] pinned host
    void** d_param_list = nullptr;         // [T] device
    void** h_param_list = nullptr;         // [T] pinned host
};

namespace {

std::atomic<int64_t> g_launches{0};
std::atomic<int64_t> g_stall_tile_p1{0};   // test hook: 1 + tile whose input copy the next step over-announces; 0: none
std::atomic<int> g_policy{0};          // 0: fastest kernel that applies; 1: general kernel only; 2: no sixteen-per-thread
                                       // kernel; 3: sixteen-per-thread kernel wherever it exists

bool valid_bits(int b) { return b == 2 || b == 3 || b == 4 || b == 8; }
bool valid_block(int b) { return b == 64 || b == 128 || b == 256 || b == 2048; }

// Signed dynamic-exponent levels (Appendix A), ascending.  With b bits, one is the
// sign and the other b-1 are E zeros, a one, and F fraction bits; a magnitude is the
// midpoint of fraction cell j of [0.1, 1] scaled by 10^-E.  Written here as the exact
// rational (2^(F+1) + 9(2j+1)) / (10^(E+1) 2^(F+1)), one binary64 division, rounded
// to binary32.  Zero and +1 complete the 2^b levels.
void de_signed_levels(int bits, std::vector<float>& y) {
    std::vector<float> pos;
    for (int E = bits - 2; E >= 0; --E) {                 // smallest decade first
        const int F = bits - 2 - E;
        const double two = (double)(1 << (F + 1));
        double ten = 10.0;
        for (int i = 0; i < E; ++i) ten *= 10.0;
        for (int j = 0; j < (1 << F); ++j)
            pos.push_back((float)((two + 9.0 * (double)(2 * j + 1)) / (ten * two)));
    }
    y.clear();
    for (size_t i = pos.size(); i-- > 0;) y.push_back(-pos[i]);
    y.push_back(0.0f);
    for (float v : pos) y.push_back(v);
    y.push_back(1.0f);
}

// y[K] | mid[K-1] = (y[k]+y[k+1])/2 | inv_gap[K-1] = 1/(y[k+1]-y[k]), all binary32.
void codebook_tables(int bits, std::vector<float>& t) {
    std::vector<float> y;
    de_signed_levels(bits, y);
    const int K = 1 << bits;
    t.assign(3 * K - 2, 0.0f);
    for (int k = 0; k < K; ++k) t[k] = y[k];
    for (int k = 0; k + 1 < K; ++k) {
        t[K + k] = 0.5f * (y[k] + y[k + 1]);
        t[2 * K - 1 + k] = 1.0f / (y[k + 1] - y[k]);
    }
}

// Unsigned codebooks of Appendix A for the baseline second-moment quantizers, ascending.
//   SOLO_V_DE            {0, 1} and 10^-E times the midpoints of the 2^F cells of [0.1, 1],
//                        E = 0..b-2 leading zero bits, one indicator bit, F = b-1-E fraction bits
//   SOLO_V_LINEAR        k / (2^b - 1), k = 0..2^b-1
//   SOLO_V_LINEAR_NOZERO k / 2^b, k = 1..2^b
void unsigned_levels(int kind, int bits, std::vector<float>& y) {
    const int K = 1 << bits;
    y.clear();
    if (kind == SOLO_V_LINEAR) {
        for (int k = 0; k < K; ++k) y.push_back((float)((double)k / (double)(K - 1)));
    } else if (kind == SOLO_V_LINEAR_NOZERO) {
        for (int k = 1; k <= K; ++k) y.push_back((float)((double)k / (double)K));
    } else {
        y.push_back(0.0f);
        for (int E = bits - 2; E >= 0; --E) {                 // smallest decade first
            const int F = bits - 1 - E;
            const double two = (double)(1 << (F + 1));
            double ten = 10.0;
            for (int i = 0; i < E; ++i) ten *= 10.0;
            for (int j = 0; j < (1 << F); ++j)
                y.push_back((float)((two + 9.0 * (double)(2 * j + 1)) / (ten * two)));
        }
        y.push_back(1.0f);
    }
}

// The three baseline tables back to back, kind = 1, 2, 3: y[K] | mid[K-1] each.
constexpr int v_table_floats(int bits) { return 2 * (1 << bits) - 1; }
void baseline_v_tables(int bits, float* t) {
    const int K = 1 << bits;
    std::vector<float> y;
    for (int kind = 1; kind <= 3; ++kind, t += v_table_floats(bits)) {
        unsigned_levels(kind, bits, y);
        for (int k = 0; k < K; ++k) t[k] = y[k];
        for (int k = 0; k + 1 < K; ++k) t[K + k] = 0.5f * (y[k] + y[k + 1]);
    }
}

__global__ void fill_f32(float* p, int64_t n, float v) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n;
         i += (int64_t)gridDim.x * blockDim.x)
        p[i] = v;
}

int sm_count(int device) {
    static std::mutex mu;
    static int cached[64];
    static bool have[64];
    std::lock_guard<std::mutex> lk(mu);
    if (device < 0 || device >= 64) return 148;
    if (!have[device]) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || v <= 0)
            v = 148;
        cached[device] = v;
        have[device] = true;
    }
    return cached[device];
}

int check_hyper(const solo_hyper_t* h, int64_t step) {
    if (!h || step < 1) return SOLO_EINVAL;
    auto unit = [](float b) { return b >= 0.0f && b < 1.0f; };
    if (!unit(h->beta1) || !unit(h->beta2) || !unit(h->p_quantile) || !unit(h->fixed_alpha)) return SOLO_EINVAL;
    if (!(h->eps >= 0.0f) || !std::isfinite(h->lr) || !std::isfinite(h->weight_decay)) return SOLO_EINVAL;
    if (h->param_dtype != 0 && h->param_dtype != 1) return SOLO_EINVAL;
    if (h->param_round != 0 && h->param_round != 1) return SOLO_EINVAL;
    if (h->v_codebook < SOLO_V_LOG || h->v_codebook > SOLO_V_LINEAR_NOZERO) return SOLO_EINVAL;
    return SOLO_OK;
}

// Bias corrections in binary64, rounded once; everything else is the caller's binary32.
void reduce_hyper(const solo_hyper_t* h, int64_t step, int block, StepArgs& a) {
    const double t = (double)step;
    const double bc1 = h->bias_correction ? 1.0 - std::pow((double)h->beta1, t) : 1.0;
    const double bc2 = h->bias_correction ? 1.0 - std::pow((double)h->beta2, t) : 1.0;
    a.beta1 = h->beta1;
    a.beta2 = h->beta2;
    a.omb1 = 1.0f - h->beta1;
    a.omb2 = 1.0f - h->beta2;
    a.step_size = (float)((double)h->lr / bc1);
    a.inv_sqrt_bc2 = (float)(1.0 / std::sqrt(bc2));
    a.eps = h->eps;
    a.decay = h->adamw ? (float)(1.0 - (double)h->lr * (double)h->weight_decay) : 1.0f;
    a.weight_decay = h->weight_decay;
    a.p_quantile = h->p_quantile;
    a.fixed_alpha = (h->fixed_alpha > 0.0f && h->fixed_alpha < 1.0f) ? h->fixed_alpha : 0.0f;
    a.l2 = (!h->adamw && h->weight_decay != 0.0f) ? 1 : 0;
    a.belief = h->belief ? 1 : 0;
    a.round_m = h->round_m ? 1 : 0;
    a.round_v = h->round_v ? 1 : 0;
    a.param_bf16 = h->param_dtype;
    a.param_sr = (h->param_dtype == 1 && h->param_round) ? 1 : 0;
    a.block = block;
    int64_t k = (int64_t)std::ceil((double)h->p_quantile * (double)block);
    a.k_full = (int)std::min<int64_t>(std::max<int64_t>(k, 1), block);
    a.seed_lo = (uint32_t)h->seed;
    a.seed_hi = (uint32_t)(h->seed >> 32);
    a.step32 = (uint32_t)step;
    for (int r = 0; r < 10; ++r) {
        a.rk[2 * r] = a.seed_lo + (uint32_t)r * 0x9E3779B9u;
        a.rk[2 * r + 1] = a.seed_hi + (uint32_t)r * 0xBB67AE85u;
    }
}

int launch_kernel(solo::StepKernel k, const StepArgs& a, int device, int threads, size_t dyn_smem,
                  cudaStream_t stream) {
    int per_sm = solo::kernel_occupancy(k, dyn_smem, threads);
    if (per_sm <= 0) return SOLO_ECUDA;
    int64_t grid = std::min<int64_t>(a.total_tiles - a.tile_first, (int64_t)sm_count(device) * per_sm);
    if (grid < 1) return SOLO_EINVAL;
    void* params[] = {(void*)&a};
    cudaError_t e = cudaLaunchKernel((const void*)k, dim3((unsigned)grid), dim3((unsigned)threads), params, dyn_smem, stream);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return SOLO_ECUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return SOLO_OK;
}

int launch_step(solo_state* s, StepArgs& a, cudaStream_t stream) {
    a.debug_stall_tile_p1 = g_stall_tile_p1.exchange(0, std::memory_order_relaxed);
    const bool cta_group = s->block == 2048;
    const int policy = g_policy.load(std::memory_order_relaxed);
    const bool fast_ok = policy != 1 && a.eps >= 1e-12f &&
                         s->tiles_total < ((int64_t)1 << 31) - ((int64_t)1 << 20);   // 32-bit tile arithmetic with headroom
    // the eight-per-thread streamlined kernel has neither the baseline second-moment codebooks nor Eq. 5
    const bool streamlined = fast_ok && !a.tables_v && !a.round_m;
    const bool plain = !a.l2 && !a.belief && a.fixed_alpha == 0.0f && a.round_v && !a.tables_v && !a.round_m;
    solo::StepKernel k16 = nullptr;
    // worth its second launch only when there is work for many tiles per CTA (measured faster on the
    // 7B-shaped, the GPT-125M-shaped and the ragged set; a 1 Mi-element tensor is launch-bound)
    const bool large = s->tiles_total >= 8192;
    // p = 0.1: rank 7, 13, 26 of a block of 64, 128, 256
    const bool rank16 = (s->block == 64 && a.k_full == 7) || (s->block == 128 && a.k_full == 13) ||
                        (s->block == 256 && a.k_full == 26);
    // (a fixed base or a baseline codebook needs no quantile, so any p goes with them)
    if (fast_ok && ((policy == 0 && large) || policy == 3) && (rank16 || a.fixed_alpha > 0.0f || a.tables_v))
        k16 = solo::fast16_kernel(s->bits_m, s->bits_v, s->block, a.param_bf16 != 0,
                                  plain ? 0 : (a.tables_v || a.round_m) ? 2 : 1);
    if (k16) {
        // full tiles by the sixteen-per-thread kernel, whatever it leaves (tails, tensors that are
        // not 16-byte aligned) by the streamlined kernel, or by the general one where that has no path
        int rc = launch_kernel(k16, a, s->device, solo::CTA16, solo::fast16_kernel_smem(s->bits_m, s->bits_v, s->block, a.param_bf16 != 0), stream);
        if (rc) return rc;
        const bool all_full = !a.param_list && s->num_tensors == 1 && s->numel[0] % solo::TILE == 0;
        if (all_full) return SOLO_OK;
        a.only_partial = 1;
    }
    solo::StepKernel k = nullptr;
    if (streamlined) k = solo::fast_kernel(s->bits_m, s->bits_v, s->block, a.param_bf16 != 0, plain);
    size_t dyn_smem = k ? solo::fast_kernel_smem(s->bits_m, s->bits_v) : 0;
    if (!k) k = solo::step_kernel(s->bits_m, s->bits_v, cta_group);
    if (!k) return SOLO_EINVAL;
    return launch_kernel(k, a, s->device, solo::CTA, dyn_smem, stream);
}

void fill_state_args(const solo_state* s, StepArgs& a) {
    const int T = s->num_tensors;
    a.numel = s->geom;
    a.block_start = s->geom + T;
    a.tile_start = s->geom + T + (T + 1);
    a.num_tensors = T;
    a.total_tiles = s->tiles_total;
    a.codes_m = s->codes_m;
    a.codes_v = s->codes_v;
    a.scale_m = s->scale_m;
    a.scale_v = s->scale_v;
    a.alpha = s->alpha;
    a.tables = s->tables_m;
    a.status = s->status;
    a.origin_id = s->origin_id;
    a.origin_ctr = s->origin_ctr;
}

// Second-moment quantizer of this step; the state remembers it for solo_dequant.
void select_v_codebook(solo_state* s, const solo_hyper_t* h, StepArgs& a) {
    a.tables_v = h->v_codebook == SOLO_V_LOG
                     ? nullptr
                     : s->tables_v + (size_t)(h->v_codebook - 1) * v_table_floats(s->bits_v);
    s->v_codebook = h->v_codebook;
}

bool on_state_device(const solo_state* s) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == s->device;
}

// ---------------------------------------------------------------------------
// Fixed scratch of the allocation-free entry point: per device, held until exit.
//   int64 numel[MAX] | block_start[MAX+1] | tile_start[MAX+1]   then
//   float tables[3*256-2] (y | mid | 1/gap of the first-moment codebook)   then
//   float tables_v[2*256-1] (y | mid of a baseline second-moment codebook)   then   int status
// ---------------------------------------------------------------------------
constexpr int STATIC_MAX_T = SOLO_STATIC_MAX_TENSORS;
constexpr size_t STATIC_GEOM_BYTES = (size_t)(3 * STATIC_MAX_T + 2) * sizeof(int64_t);
constexpr size_t STATIC_TABLE_BYTES = (size_t)(3 * 256 - 2) * sizeof(float);
constexpr size_t STATIC_VTABLE_BYTES = (size_t)(2 * 256 - 1) * sizeof(float);
constexpr size_t STATIC_STATUS_OFF =
    (STATIC_GEOM_BYTES + STATIC_TABLE_BYTES + STATIC_VTABLE_BYTES + 15) / 16 * 16;
constexpr size_t STATIC_BYTES = STATIC_STATUS_OFF + 16;
static_assert(STATIC_BYTES <= 32 * 1024, "documented size of the fixed scratch");

static __device__ __align__(256) unsigned char g_static_scratch[STATIC_BYTES];
// Zeros, never written: the default position in the random stream of every tensor of a
// solo_multi_step_static call (read as the int32 and as the int64 array of StepArgs).
static __device__ __align__(256) int64_t g_static_zero_origin[STATIC_MAX_T];

// Device address of g_static_scratch on the current device (the symbol's name is only a
// host-side handle).  Looked up once per device, with that device current.
int static_scratch(int device, unsigned char** out, const int64_t** zeros_out = nullptr) {
    static std::mutex mu;
    static unsigned char* ptr[64];
    static const int64_t* zeros[64];
    if (device < 0 || device >= 64) return SOLO_EINVAL;
    std::lock_guard<std::mutex> lk(mu);
    if (!ptr[device]) {
        void *p = nullptr, *z = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p ||
            cudaGetSymbolAddress(&z, g_static_zero_origin) != cudaSuccess || !z) {
            cudaGetLastError();
            return SOLO_ECUDA;
        }
        ptr[device] = (unsigned char*)p;
        zeros[device] = (const int64_t*)z;
    }
    *out = ptr[device];
    if (zeros_out) *zeros_out = zeros[device];
    return SOLO_OK;
}

}  // namespace

extern "C" {

int solo_state_bytes(int64_t numel, int bits_m, int bits_v, int block, size_t* out) {
    if (!out || numel < 0 || !valid_bits(bits_m) || !valid_bits(bits_v) || !valid_block(block))
        return SOLO_EINVAL;
    const int64_t nblk = (numel + block - 1) / block;
    *out = (size_t)nblk * (size_t)(block * bits_m / 8) + (size_t)nblk * (size_t)(block * bits_v / 8) +
           (size_t)nblk * 12u;
    return SOLO_OK;
}

int solo_state_create_multi(const int64_t* numel_host, int num_tensors, int bits_m, int bits_v,
                            int block, solo_state_t** out) {
    if (!out) return SOLO_EINVAL;
    *out = nullptr;
    if (!numel_host || num_tensors < 1 || !valid_bits(bits_m) || !valid_bits(bits_v) || !valid_block(block))
        return SOLO_EINVAL;
    for (int t = 0; t < num_tensors; ++t)
        if (numel_host[t] < 1) return SOLO_EINVAL;
    solo_state* s = new (std::nothrow) solo_state();
    if (!s) return SOLO_ENOMEM;
    if (cudaGetDevice(&s->device) != cudaSuccess) { delete s; return SOLO_ECUDA; }
    s->bits_m = bits_m; s->bits_v = bits_v; s->block = block; s->num_tensors = num_tensors;
    const int T = num_tensors;
    s->numel.assign(numel_host, numel_host + T);
    s->block_start.assign(T + 1, 0);
    s->tile_start.assign(T + 1, 0);
    s->elem_start.assign(T + 1, 0);
    for (int t = 0; t < T; ++t) {
        s->block_start[t + 1] = s->block_start[t] + (numel_host[t] + block - 1) / block;
        s->tile_start[t + 1] = s->tile_start[t] + (numel_host[t] + solo::TILE - 1) / solo::TILE;
        s->elem_start[t + 1] = s->elem_start[t] + numel_host[t];
    }
    s->numel_total = s->elem_start[T];
    s->nblk_total = s->block_start[T];
    s->tiles_total = s->tile_start[T];
    s->bytes_codes_m = (size_t)s->nblk_total * (size_t)(block * bits_m / 8);
    s->bytes_codes_v = (size_t)s->nblk_total * (size_t)(block * bits_v / 8);

    std::vector<int64_t> geom;
    geom.insert(geom.end(), s->numel.begin(), s->numel.end());
    geom.insert(geom.end(), s->block_start.begin(), s->block_start.end());
    geom.insert(geom.end(), s->tile_start.begin(), s->tile_start.end());
    geom.insert(geom.end(), s->elem_start.begin(), s->elem_start.end());
    std::vector<float> tm, tv;
    codebook_tables(bits_m, tm);
    tv.assign(3 * v_table_floats(bits_v), 0.0f);
    baseline_v_tables(bits_v, tv.data());

    bool ok = true;
    auto alloc = [&](void** p, size_t bytes) {
        if (ok && cudaMalloc(p, bytes ? bytes : 1) != cudaSuccess) { ok = false; cudaGetLastError(); }
    };
    // 16 bytes of slack after the codes: the streamlined kernel copies a tile's codes in
    // 16-byte pieces starting at the 16-byte boundary at or below them
    alloc((void**)&s->codes_m, s->bytes_codes_m + 16);
    alloc((void**)&s->codes_v, s->bytes_codes_v + 16);
    // the three per-block arrays are allocated in multiples of 16 bytes (the streamlined kernel
    // copies them in 16-byte pieces)
    const size_t scal_bytes = ((size_t)s->nblk_total + 3) / 4 * 16;
    alloc((void**)&s->scale_m, scal_bytes);
    alloc((void**)&s->scale_v, scal_bytes);
    alloc((void**)&s->alpha, scal_bytes);
    alloc((void**)&s->geom, geom.size() * 8);
    alloc((void**)&s->tables_m, tm.size() * 4);
    alloc((void**)&s->tables_v, tv.size() * 4);
    alloc((void**)&s->status, 4);
    alloc((void**)&s->origin_id, (size_t)T * 4);
    alloc((void**)&s->origin_ctr, (size_t)T * 8);
    if (!ok) { solo_state_destroy(s); return SOLO_ENOMEM; }
    cudaError_t e = cudaSuccess;
    auto chk = [&](cudaError_t r) { if (e == cudaSuccess) e = r; };
    chk(cudaMemset(s->codes_m, 0, s->bytes_codes_m + 16));
    chk(cudaMemset(s->codes_v, 0, s->bytes_codes_v + 16));
    chk(cudaMemset(s->scale_m, 0, scal_bytes));
    chk(cudaMemset(s->scale_v, 0, scal_bytes));
    chk(cudaMemset(s->alpha, 0, scal_bytes));
    chk(cudaMemset(s->status, 0, 4));
    chk(cudaMemset(s->origin_id, 0, (size_t)T * 4));
    chk(cudaMemset(s->origin_ctr, 0, (size_t)T * 8));
    chk(cudaMemcpy(s->geom, geom.data(), geom.size() * 8, cudaMemcpyHostToDevice));
    chk(cudaMemcpy(s->tables_m, tm.data(), tm.size() * 4, cudaMemcpyHostToDevice));
    chk(cudaMemcpy(s->tables_v, tv.data(), tv.size() * 4, cudaMemcpyHostToDevice));
    if (e == cudaSuccess) {
        fill_f32<<<1024, 256>>>(s->alpha, s->nblk_total, 0.5f);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        chk(cudaGetLastError());
        chk(cudaDeviceSynchronize());
    }
    if (e != cudaSuccess) { solo_state_destroy(s); return SOLO_ECUDA; }
    *out = s;
    return SOLO_OK;
}

int solo_state_create(int64_t numel, int bits_m, int bits_v, int block, solo_state_t** out) {
    return solo_state_create_multi(&numel, 1, bits_m, bits_v, block, out);
}

int solo_state_destroy(solo_state_t* s) {
    if (!s) return SOLO_OK;
    cudaDeviceSynchronize();
    if (s->pipe) {
        HostPipe* hp = s->pipe;
        for (int i = 0; i < HostPipe::SLOTS; ++i) {
            if (hp->stream[i]) cudaStreamDestroy(hp->stream[i]);
            if (hp->done[i]) cudaEventDestroy(hp->done[i]);
            if (hp->d_grad[i]) cudaFree(hp->d_grad[i]);
            if (hp->d_grad_list[i]) cudaFree(hp->d_grad_list[i]);
            if (hp->h_grad_list[i]) cudaFreeHost(hp->h_grad_list[i]);
        }
        if (hp->start) cudaEventDestroy(hp->start);
        if (hp->d_param_list) cudaFree(hp->d_param_list);
        if (hp->h_param_list) cudaFreeHost(hp->h_param_list);
        delete hp;
        s->pipe = nullptr;
    }
    void* ptrs[] = {s->codes_m, s->codes_v, s->scale_m, s->scale_v, s->alpha,
                    s->geom, s->tables_m, s->tables_v, s->status, s->origin_id, s->origin_ctr};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    delete s;
    return SOLO_OK;
}

int solo_state_set_origin(solo_state_t* s, const int32_t* stream_id_host, const int64_t* elem_offset_host) {
    if (!s) return SOLO_EINVAL;
    if (!on_state_device(s)) return SOLO_ESTATE;
    const int T = s->num_tensors;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return SOLO_ECUDA; }   // steps in flight read the arrays
    std::vector<int32_t> id((size_t)T);
    std::vector<int64_t> ctr((size_t)T);
    for (int t = 0; t < T; ++t) {
        const int32_t stream = stream_id_host ? stream_id_host[t] : t;
        const int64_t off = elem_offset_host ? elem_offset_host[t] : 0;
        // a shard starts on a block boundary of its tensor; the stream id shares a 32-bit word with the purpose
        if (off < 0 || off % s->block != 0 || stream < 0 || stream >= (1 << 30)) return SOLO_EINVAL;
        id[t] = stream - t;
        ctr[t] = off / 8;
    }
    if (cudaMemcpy(s->origin_id, id.data(), (size_t)T * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(s->origin_ctr, ctr.data(), (size_t)T * 8, cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError();
        return SOLO_ECUDA;
    }
    return SOLO_OK;
}

int solo_step(void* param_dev, const void* grad_dev, solo_state_t* s, const solo_hyper_t* hyper,
              int64_t step, void* stream) {
    if (!param_dev || !grad_dev || !s) return SOLO_EINVAL;
    int rc = check_hyper(hyper, step);
    if (rc) return rc;
    if (s->num_tensors != 1 || !on_state_device(s)) return SOLO_ESTATE;
    if ((((uintptr_t)param_dev) | ((uintptr_t)grad_dev)) & 15u) return SOLO_EALIGN;
    StepArgs a;
    std::memset(&a, 0, sizeof(a));
    fill_state_args(s, a);
    reduce_hyper(hyper, step, s->block, a);
    select_v_codebook(s, hyper, a);
    a.param_single = param_dev;
    a.grad_single = grad_dev;
    return launch_step(s, a, (cudaStream_t)stream);
}

int solo_multi_step(const solo_tensor_list_t* list, const solo_hyper_t* hyper, int64_t step,
                    void* stream) {
    if (!list || !list->state || !list->param || !list->grad) return SOLO_EINVAL;
    int rc = check_hyper(hyper, step);
    if (rc) return rc;
    solo_state* s = list->state;
    if (list->num_tensors != s->num_tensors || !on_state_device(s)) return SOLO_ESTATE;
    StepArgs a;
    std::memset(&a, 0, sizeof(a));
    fill_state_args(s, a);
    reduce_hyper(hyper, step, s->block, a);
    select_v_codebook(s, hyper, a);
    a.param_list = list->param;
    a.grad_list = list->grad;
    a.numel_check = list->numel;
    return launch_step(s, a, (cudaStream_t)stream);
}

namespace {

// Creates (or, for another chunk size, re-creates) the staging of solo_multi_step_host.
int host_pipe_prepare(solo_state* s, int64_t chunk_tiles) {
    HostPipe* hp = s->pipe;
    if (hp && hp->chunk_tiles == chunk_tiles) return SOLO_OK;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return SOLO_ECUDA; }
    if (!hp) {
        hp = new (std::nothrow) HostPipe();
        if (!hp) return SOLO_ENOMEM;
        s->pipe = hp;
        const size_t list_bytes = (size_t)s->num_tensors * sizeof(void*);
        bool ok = cudaEventCreateWithFlags(&hp->start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaMalloc((void**)&hp->d_param_list, list_bytes) == cudaSuccess &&
                  cudaMallocHost((void**)&hp->h_param_list, list_bytes) == cudaSuccess;
        for (int i = 0; ok && i < HostPipe::SLOTS; ++i)
            ok = cudaStreamCreateWithFlags(&hp->stream[i], cudaStreamNonBlocking) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp->done[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaMalloc((void**)&hp->d_grad_list[i], list_bytes) == cudaSuccess &&
                 cudaMallocHost((void**)&hp->h_grad_list[i], list_bytes) == cudaSuccess;
        if (!ok) { cudaGetLastError(); return SOLO_ENOMEM; }   // what exists is freed with the state
    }
    for (int i = 0; i < HostPipe::SLOTS; ++i) {
        if (hp->d_grad[i]) cudaFree(hp->d_grad[i]);
        hp->d_grad[i] = nullptr;
    }
    hp->chunk_tiles = 0;
    const size_t slot_bytes = (size_t)chunk_tiles * (solo::TILE * 2 + 16);
    for (int i = 0; i < HostPipe::SLOTS; ++i)
        if (cudaMalloc((void**)&hp->d_grad[i], slot_bytes) != cudaSuccess) { cudaGetLastError(); return SOLO_ENOMEM; }
    hp->chunk_tiles = chunk_tiles;
    return SOLO_OK;
}

}  // namespace

int solo_multi_step_host(const solo_host_list_t* list, const solo_hyper_t* hyper, int64_t step,
                         void* stream_) {
    if (!list || !list->state || !list->param_dev || !list->grad_host || !list->numel) return SOLO_EINVAL;
    int rc = check_hyper(hyper, step);
    if (rc) return rc;
    solo_state* s = list->state;
    const int T = s->num_tensors;
    if (list->num_tensors != T || !on_state_device(s)) return SOLO_ESTATE;
    if (list->chunk_elems < 0) return SOLO_EINVAL;
    const int psz = hyper->param_dtype == 1 ? 2 : 4;
    for (int t = 0; t < T; ++t) {
        if (list->numel[t] != s->numel[t]) return SOLO_ESTATE;
        if (!list->param_dev[t] || !list->grad_host[t] || (list->param_out_host && !list->param_out_host[t]))
            return SOLO_EINVAL;
        if (((uintptr_t)list->param_dev[t]) & 15u) return SOLO_EALIGN;
    }
    const int64_t chunk_elems = list->chunk_elems ? list->chunk_elems : (int64_t)16 << 20;
    const int64_t chunk_tiles = std::max<int64_t>(1, chunk_elems / solo::TILE);
    rc = host_pipe_prepare(s, chunk_tiles);
    if (rc) return rc;
    HostPipe* hp = s->pipe;
    cudaStream_t user = (cudaStream_t)stream_;
    bool ok = true;
    auto chk = [&](cudaError_t e) { ok = ok && e == cudaSuccess; };

    // the call before this one may still be using the pinned pointer arrays and the slots
    for (int i = 0; i < HostPipe::SLOTS; ++i) chk(cudaEventSynchronize(hp->done[i]));
    for (int t = 0; t < T; ++t) hp->h_param_list[t] = list->param_dev[t];
    chk(cudaMemcpyAsync(hp->d_param_list, hp->h_param_list, (size_t)T * sizeof(void*), cudaMemcpyHostToDevice, user));
    chk(cudaEventRecord(hp->start, user));
    for (int i = 0; i < HostPipe::SLOTS; ++i) chk(cudaStreamWaitEvent(hp->stream[i], hp->start, 0));
    if (!ok) { cudaGetLastError(); return SOLO_ECUDA; }

    StepArgs base;
    std::memset(&base, 0, sizeof(base));
    fill_state_args(s, base);
    reduce_hyper(hyper, step, s->block, base);
    select_v_codebook(s, hyper, base);
    base.param_list = hp->d_param_list;

    int tensor = 0;
    int64_t chunk = 0;
    for (int64_t first = 0; first < s->tiles_total; first += chunk_tiles, ++chunk) {
        const int64_t last = std::min<int64_t>(s->tiles_total, first + chunk_tiles);
        const int slot = (int)(chunk % HostPipe::SLOTS);
        cudaStream_t st = hp->stream[slot];
        if (chunk >= HostPipe::SLOTS) chk(cudaEventSynchronize(hp->done[slot]));   // its pinned list is free again
        while (s->tile_start[tensor + 1] <= first) ++tensor;
        const int tensor_first = tensor;
        // upload: one piece per tensor that the chunk touches, each from a 16-byte boundary of the slot
        size_t off = 0;
        int t = tensor;
        for (; t < T && s->tile_start[t] < last; ++t) {
            const int64_t e_lo = (std::max<int64_t>(s->tile_start[t], first) - s->tile_start[t]) * solo::TILE;
            const int64_t e_hi = std::min<int64_t>(s->numel[t],
                                                   (std::min<int64_t>(s->tile_start[t + 1], last) - s->tile_start[t]) * solo::TILE);
            const size_t bytes = (size_t)(e_hi - e_lo) * 2;
            chk(cudaMemcpyAsync(hp->d_grad[slot] + off, (const char*)list->grad_host[t] + e_lo * 2, bytes,
                                cudaMemcpyHostToDevice, st));
            // the kernel indexes gradients by the element's position in its tensor
            hp->h_grad_list[slot][t] = (void*)((uintptr_t)hp->d_grad[slot] + off - (uintptr_t)(e_lo * 2));
            off += (bytes + 15) / 16 * 16;
        }
        const int t_end = t;
        chk(cudaMemcpyAsync(hp->d_grad_list[slot] + tensor_first, hp->h_grad_list[slot] + tensor_first,
                            (size_t)(t_end - tensor_first) * sizeof(void*), cudaMemcpyHostToDevice, st));
        if (!ok) break;
        StepArgs a = base;
        a.grad_list = (const void* const*)hp->d_grad_list[slot];
        a.tile_first = first;
        a.total_tiles = last;
        rc = launch_step(s, a, st);
        if (rc) break;
        if (list->param_out_host) {
            for (t = tensor_first; t < t_end; ++t) {
                const int64_t e_lo = (std::max<int64_t>(s->tile_start[t], first) - s->tile_start[t]) * solo::TILE;
                const int64_t e_hi = std::min<int64_t>(s->numel[t],
                                                       (std::min<int64_t>(s->tile_start[t + 1], last) - s->tile_start[t]) * solo::TILE);
                chk(cudaMemcpyAsync((char*)list->param_out_host[t] + e_lo * psz, (const char*)list->param_dev[t] + e_lo * psz,
                                    (size_t)(e_hi - e_lo) * psz, cudaMemcpyDeviceToHost, st));
            }
        }
        chk(cudaEventRecord(hp->done[slot], st));
    }
    // the caller's stream continues after every slot's last chunk, also when something failed
    for (int i = 0; i < HostPipe::SLOTS; ++i) {
        cudaEventRecord(hp->done[i], hp->stream[i]);
        cudaStreamWaitEvent(user, hp->done[i], 0);
    }
    if (rc) return rc;
    if (!ok) { cudaGetLastError(); return SOLO_ECUDA; }
    return SOLO_OK;
}

int solo_multi_step_static(int32_t num_tensors, void* const* param_dev, const void* const* grad_dev,
                           const int64_t* numel_host, const solo_raw_state_t* st,
                           const solo_hyper_t* hyper, int64_t step, void* stream_) {
    if (!param_dev || !grad_dev || !numel_host || !st || num_tensors < 1) return SOLO_EINVAL;
    if (num_tensors > STATIC_MAX_T) return SOLO_ELIMIT;
    if (!valid_bits(st->bits_m) || !valid_bits(st->bits_v) || !valid_block(st->block)) return SOLO_EINVAL;
    if (!st->codes_m || !st->codes_v || !st->scale_m || !st->scale_v || !st->alpha) return SOLO_EINVAL;
    if ((((uintptr_t)st->codes_m) | ((uintptr_t)st->codes_v) | ((uintptr_t)st->scale_m) |
         ((uintptr_t)st->scale_v) | ((uintptr_t)st->alpha)) & 15u)
        return SOLO_EALIGN;
    int rc = check_hyper(hyper, step);
    if (rc) return rc;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return SOLO_ECUDA; }
    unsigned char* scratch = nullptr;
    const int64_t* zero_origin = nullptr;
    rc = static_scratch(device, &scratch, &zero_origin);
    if (rc) return rc;
    cudaStream_t stream = (cudaStream_t)stream_;
    // the tables below are copied from this call's stack: a captured copy would read a dead frame at replay
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) { cudaGetLastError(); return SOLO_ECUDA; }
    if (cap != cudaStreamCaptureStatusNone) return SOLO_EINVAL;

    // geometry and codebook tables, built in fixed-size host arrays (no device allocation)
    const int T = num_tensors, block = st->block;
    int64_t geom[3 * STATIC_MAX_T + 2];
    int64_t* numel = geom;
    int64_t* block_start = geom + T;
    int64_t* tile_start = geom + T + (T + 1);
    block_start[0] = 0;
    tile_start[0] = 0;
    for (int t = 0; t < T; ++t) {
        if (numel_host[t] < 1) return SOLO_EINVAL;
        numel[t] = numel_host[t];
        block_start[t + 1] = block_start[t] + (numel_host[t] + block - 1) / block;
        tile_start[t + 1] = tile_start[t] + (numel_host[t] + solo::TILE - 1) / solo::TILE;
    }
    float tables[3 * 256 - 2];
    {
        std::vector<float> tm;                       // host memory only
        codebook_tables(st->bits_m, tm);
        std::memcpy(tables, tm.data(), tm.size() * sizeof(float));
    }
    float tables_v[2 * 256 - 1];
    const bool vtab = hyper->v_codebook != SOLO_V_LOG;
    if (vtab) {
        float all[3 * (2 * 256 - 1)];
        baseline_v_tables(st->bits_v, all);             // std::vector inside: host memory only
        std::memcpy(tables_v, all + (size_t)(hyper->v_codebook - 1) * v_table_floats(st->bits_v),
                    (size_t)v_table_floats(st->bits_v) * sizeof(float));
    }
    const size_t geom_bytes = (size_t)(3 * T + 2) * sizeof(int64_t);
    const size_t table_bytes = (size_t)(3 * (1 << st->bits_m) - 2) * sizeof(float);
    int64_t* d_geom = (int64_t*)scratch;
    float* d_tables = (float*)(scratch + STATIC_GEOM_BYTES);
    float* d_tables_v = (float*)(scratch + STATIC_GEOM_BYTES + STATIC_TABLE_BYTES);
    int* d_status = (int*)(scratch + STATIC_STATUS_OFF);
    // pageable sources: both copies are staged before cudaMemcpyAsync returns
    if (cudaMemcpyAsync(d_geom, geom, geom_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(d_tables, tables, table_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        (vtab && cudaMemcpyAsync(d_tables_v, tables_v, (size_t)v_table_floats(st->bits_v) * sizeof(float),
                                 cudaMemcpyHostToDevice, stream) != cudaSuccess) ||
        cudaMemsetAsync(d_status, 0, 16, stream) != cudaSuccess) {
        cudaGetLastError();
        return SOLO_ECUDA;
    }

    solo_state tmp;                                   // host-side description only; owns nothing
    tmp.device = device;
    tmp.bits_m = st->bits_m; tmp.bits_v = st->bits_v; tmp.block = block; tmp.num_tensors = T;
    tmp.tiles_total = tile_start[T];
    tmp.nblk_total = block_start[T];
    StepArgs a;
    std::memset(&a, 0, sizeof(a));
    a.numel = d_geom;
    a.block_start = d_geom + T;
    a.tile_start = d_geom + T + (T + 1);
    a.num_tensors = T;
    a.total_tiles = tmp.tiles_total;
    a.codes_m = (uint8_t*)st->codes_m;
    a.codes_v = (uint8_t*)st->codes_v;
    a.scale_m = st->scale_m;
    a.scale_v = st->scale_v;
    a.alpha = st->alpha;
    a.tables = d_tables;
    a.tables_v = vtab ? d_tables_v : nullptr;
    a.status = d_status;
    a.origin_id = (const int32_t*)zero_origin;
    a.origin_ctr = zero_origin;
    reduce_hyper(hyper, step, block, a);
    a.param_list = param_dev;
    a.grad_list = grad_dev;
    a.numel_check = nullptr;
    return launch_step(&tmp, a, stream);
}

int solo_static_status(int* status_out, void* stream_) {
    if (!status_out) return SOLO_EINVAL;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return SOLO_ECUDA; }
    unsigned char* scratch = nullptr;
    int rc = static_scratch(device, &scratch);
    if (rc) return rc;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (cudaMemcpyAsync(status_out, scratch + STATIC_STATUS_OFF, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
        cudaGetLastError();
        return SOLO_ECUDA;
    }
    return SOLO_OK;
}

int solo_debug_stall_copy(int64_t tile) {
    if (tile < 0) return SOLO_EINVAL;
    g_stall_tile_p1.store(tile + 1, std::memory_order_relaxed);
    return SOLO_OK;
}

int solo_dequant(const solo_state_t* s, int which, float* out_dev, void* stream) {
    if (!s || !out_dev || (which != 0 && which != 1)) return SOLO_EINVAL;
    if (!on_state_device(s)) return SOLO_ESTATE;
    solo::DequantArgs a;
    std::memset(&a, 0, sizeof(a));
    const int T = s->num_tensors;
    a.numel = s->geom;
    a.block_start = s->geom + T;
    a.tile_start = s->geom + T + (T + 1);
    a.elem_start = s->geom + T + 2 * (T + 1);
    a.num_tensors = T;
    a.total_tiles = s->tiles_total;
    a.codes = which == 0 ? s->codes_m : s->codes_v;
    a.scale = which == 0 ? s->scale_m : s->scale_v;
    a.alpha = s->alpha;
    a.tables = s->tables_m;
    a.out = out_dev;
    a.block = s->block;
    a.which = which;
    if (which == 1 && s->v_codebook != SOLO_V_LOG) {          // level table times scale
        a.tables = s->tables_v + (size_t)(s->v_codebook - 1) * v_table_floats(s->bits_v);
        a.which = 0;
    }
    const int bits = which == 0 ? s->bits_m : s->bits_v;
    int64_t grid = std::min<int64_t>(s->tiles_total, (int64_t)sm_count(s->device) * 8);
    cudaError_t e = solo::launch_dequant(bits, a, (unsigned)grid, (cudaStream_t)stream);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return SOLO_ECUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return SOLO_OK;
}

int solo_state_raw(const solo_state_t* s, int which, void** dev_ptr, size_t* bytes) {
    if (!s || !dev_ptr || !bytes) return SOLO_EINVAL;
    switch (which) {
        case 0: *dev_ptr = s->codes_m; *bytes = s->bytes_codes_m; break;
        case 1: *dev_ptr = s->codes_v; *bytes = s->bytes_codes_v; break;
        case 2: *dev_ptr = s->scale_m; *bytes = (size_t)s->nblk_total * 4; break;
        case 3: *dev_ptr = s->scale_v; *bytes = (size_t)s->nblk_total * 4; break;
        case 4: *dev_ptr = s->alpha; *bytes = (size_t)s->nblk_total * 4; break;
        default: return SOLO_EINVAL;
    }
    return SOLO_OK;
}

int solo_state_info(const solo_state_t* s, int64_t* numel, int64_t* num_blocks, int32_t* num_tensors,
                    int32_t* bits_m, int32_t* bits_v, int32_t* block) {
    if (!s) return SOLO_EINVAL;
    if (numel) *numel = s->numel_total;
    if (num_blocks) *num_blocks = s->nblk_total;
    if (num_tensors) *num_tensors = s->num_tensors;
    if (bits_m) *bits_m = s->bits_m;
    if (bits_v) *bits_v = s->bits_v;
    if (block) *block = s->block;
    return SOLO_OK;
}

namespace {
constexpr char CKPT_MAGIC[8] = {'S', 'O', 'L', 'O', 'S', 'T', '1', 0};
size_t pad16(size_t n) { return (n + 15) / 16 * 16; }
size_t ckpt_header_bytes(int T) { return pad16(8 + 6 * 4 + 8 + (size_t)T * 8); }
struct CkptPart { void* dev; size_t bytes; };
void ckpt_parts(const solo_state* s, CkptPart (&p)[5]) {
    p[0] = {s->codes_m, s->bytes_codes_m};
    p[1] = {s->codes_v, s->bytes_codes_v};
    p[2] = {s->scale_m, (size_t)s->nblk_total * 4};
    p[3] = {s->scale_v, (size_t)s->nblk_total * 4};
    p[4] = {s->alpha, (size_t)s->nblk_total * 4};
}
size_t ckpt_bytes(const solo_state* s) {
    CkptPart p[5];
    ckpt_parts(s, p);
    size_t n = ckpt_header_bytes(s->num_tensors);
    for (const CkptPart& q : p) n += pad16(q.bytes);
    return n;
}
}  // namespace

int solo_state_export_bytes(const solo_state_t* s, size_t* out) {
    if (!s || !out) return SOLO_EINVAL;
    *out = ckpt_bytes(s);
    return SOLO_OK;
}

int solo_state_export(const solo_state_t* s, void* host_dst, size_t bytes, void* stream_) {
    if (!s || !host_dst) return SOLO_EINVAL;
    if (bytes < ckpt_bytes(s)) return SOLO_EINVAL;
    if (!on_state_device(s)) return SOLO_ESTATE;
    cudaStream_t stream = (cudaStream_t)stream_;
    unsigned char* dst = (unsigned char*)host_dst;
    const int T = s->num_tensors;
    std::memset(dst, 0, ckpt_header_bytes(T));
    std::memcpy(dst, CKPT_MAGIC, 8);
    const int32_t head[6] = {s->bits_m, s->bits_v, s->block, T, s->v_codebook, 0};
    std::memcpy(dst + 8, head, sizeof(head));
    std::memcpy(dst + 32, &s->nblk_total, 8);
    std::memcpy(dst + 40, s->numel.data(), (size_t)T * 8);
    size_t off = ckpt_header_bytes(T);
    CkptPart p[5];
    ckpt_parts(s, p);
    for (const CkptPart& q : p) {
        if (cudaMemcpyAsync(dst + off, q.dev, q.bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess) {
            cudaGetLastError();
            return SOLO_ECUDA;
        }
        std::memset(dst + off + q.bytes, 0, pad16(q.bytes) - q.bytes);   // padding, outside the copy
        off += pad16(q.bytes);
    }
    if (cudaStreamSynchronize(stream) != cudaSuccess) { cudaGetLastError(); return SOLO_ECUDA; }
    return SOLO_OK;
}

int solo_state_import(solo_state_t* s, const void* host_src, size_t bytes, void* stream_) {
    if (!s || !host_src) return SOLO_EINVAL;
    const unsigned char* src = (const unsigned char*)host_src;
    if (bytes < 40 || std::memcmp(src, CKPT_MAGIC, 8) != 0) return SOLO_EINVAL;
    int32_t head[6];
    int64_t nblk = 0;
    std::memcpy(head, src + 8, sizeof(head));
    std::memcpy(&nblk, src + 32, 8);
    if (head[0] != s->bits_m || head[1] != s->bits_v || head[2] != s->block || head[3] != s->num_tensors ||
        nblk != s->nblk_total)
        return SOLO_ESTATE;
    if (head[4] < SOLO_V_LOG || head[4] > SOLO_V_LINEAR_NOZERO) return SOLO_EINVAL;
    if (bytes < ckpt_bytes(s)) return SOLO_EINVAL;
    if (std::memcmp(src + 40, s->numel.data(), (size_t)s->num_tensors * 8) != 0) return SOLO_ESTATE;
    if (!on_state_device(s)) return SOLO_ESTATE;
    cudaStream_t stream = (cudaStream_t)stream_;
    size_t off = ckpt_header_bytes(s->num_tensors);
    CkptPart p[5];
    ckpt_parts(s, p);
    for (const CkptPart& q : p) {
        if (cudaMemcpyAsync(q.dev, src + off, q.bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) {
            cudaGetLastError();
            return SOLO_ECUDA;
        }
        off += pad16(q.bytes);
    }
    if (cudaStreamSynchronize(stream) != cudaSuccess) { cudaGetLastError(); return SOLO_ECUDA; }
    s->v_codebook = head[4];
    return SOLO_OK;
}

int solo_state_status(solo_state_t* s, int* status_out) {
    if (!s || !status_out) return SOLO_EINVAL;
    if (!on_state_device(s)) return SOLO_ESTATE;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return SOLO_ECUDA; }
    if (cudaMemcpy(status_out, s->status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return SOLO_ECUDA;
    }
    return SOLO_OK;
}

int solo_codebook_m(int bits, float* levels_host) {
    if (!valid_bits(bits) || !levels_host) return SOLO_EINVAL;
    std::vector<float> y;
    de_signed_levels(bits, y);
    std::memcpy(levels_host, y.data(), y.size() * 4);
    return SOLO_OK;
}

int solo_codebook_v(int v_codebook, int bits, float* levels_host) {
    if (!valid_bits(bits) || !levels_host) return SOLO_EINVAL;
    if (v_codebook < SOLO_V_DE || v_codebook > SOLO_V_LINEAR_NOZERO) return SOLO_EINVAL;
    std::vector<float> y;
    unsigned_levels(v_codebook, bits, y);
    std::memcpy(levels_host, y.data(), y.size() * 4);
    return SOLO_OK;
}

float solo_default_beta1(int bits_m, int from_scratch) {
    if (bits_m < 2 || bits_m > 8) return 0.0f;
    auto r_median = [](int bits) {
        std::vector<float> y;
        de_signed_levels(bits, y);
        std::vector<double> r;
        for (size_t k = 0; k + 1 < y.size(); ++k) r.push_back(0.5 * ((double)y[k + 1] - (double)y[k]));
        std::sort(r.begin(), r.end());
        const size_t n = r.size();
        return n % 2 ? r[n / 2] : 0.5 * (r[n / 2 - 1] + r[n / 2]);
    };
    const int b = from_scratch ? 8 : 5;
    if (bits_m >= b) return 0.9f;
    const double c = 0.9 / 0.1 * r_median(b) / r_median(bits_m);
    const double bound = c / (1.0 + c);
    return (float)(std::floor(bound * 10.0 + 1e-9) / 10.0);
}

int solo_set_kernel_policy(int policy) {
    if (policy < 0 || policy > 3) return SOLO_EINVAL;
    g_policy.store(policy, std::memory_order_relaxed);
    return SOLO_OK;
}

int solo_debug_check_fast_log(uint32_t lo_bits, uint32_t hi_bits, float* max_excess_host,
                              float* abs_bound_host) {
    if (!max_excess_host || !abs_bound_host || lo_bits > hi_bits || lo_bits < 0x00800000u ||
        hi_bits >= 0x7F800000u)
        return SOLO_EINVAL;
    float* d = nullptr;
    if (cudaMalloc((void**)&d, 4) != cudaSuccess) { cudaGetLastError(); return SOLO_ENOMEM; }
    const float init = -1.0f;
    cudaError_t e = cudaMemcpy(d, &init, 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = solo::launch_fast_log_check(lo_bits, hi_bits, d, nullptr);
    if (e == cudaSuccess) g_launches.fetch_add(1, std::memory_order_relaxed);
    if (e == cudaSuccess) e = cudaMemcpy(max_excess_host, d, 4, cudaMemcpyDeviceToHost);
    cudaFree(d);
    if (e != cudaSuccess) { cudaGetLastError(); return SOLO_ECUDA; }
    *abs_bound_host = solo::fast_log_abs_bound();
    return SOLO_OK;
}

int64_t solo_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* solo_strerror(int status) {
    switch (status) {
        case SOLO_OK: return "ok";
        case SOLO_EINVAL: return "invalid argument";
        case SOLO_EALIGN: return "parameter or gradient pointer is not 16-byte aligned";
        case SOLO_ENOMEM: return "out of memory";
        case SOLO_ECUDA: return "CUDA call or kernel launch failed";
        case SOLO_ESTATE: return "state does not match the call";
        case SOLO_ELIMIT: return "too many tensors for solo_multi_step_static (limit SOLO_STATIC_MAX_TENSORS)";
        default: return "unknown status";
    }
}

}  // extern "C"
