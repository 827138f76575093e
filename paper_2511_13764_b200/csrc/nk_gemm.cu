// Host side of the nk_gemm C ABI: descriptor validation, the plan-time choice of
// kernel / tile / K split, TMA tensor-map encoding, and the launches.  All the
// arithmetic of the GEMM runs in the kernels included below.
#include "../../include/nk_gemm.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>

#include "aux_kernels.cuh"
#include "simt_f32.cuh"
#include "umma_bf16.cuh"
#include "umma_bf16_pair.cuh"
#include "umma_swap.cuh"
#include <atomic>

namespace nk {

// Status words, a static table per device (the module is instantiated on every device that
// loads the library).  A plan takes the next slot of the table when it is created (round robin:
// two plans share a word only when more than NK_STATUS_SLOTS plans were created in between), so a
// wait that ran out is reported by the plan whose kernel it was.  Kernels receive the slot's
// device address as a parameter; nothing is allocated.
constexpr unsigned NK_STATUS_SLOTS = 1024;
__device__ unsigned int g_status_word[NK_STATUS_SLOTS];
static std::atomic<unsigned> g_next_status_slot{0};

enum Variant { V_NAIVE = 0, V_SIMT = 1, V_UMMA = 2, V_SKINNY = 3, V_SPLIT3 = 4, V_SMALL = 5, V_SWAP = 6 };

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace nk

struct nk_gemm_s {
    nk_gemm_desc_t d;
    int variant;
    int sm_count;
    // UMMA
    int bn, stages, splits, group_m;
    int swap_mp;           // swap-AB skinny kernel: M rounded up to 16, 32 or 64
    bool serpentine;       // raster: odd groups of M tiles sweep N backwards
    bool k_serpentine;     // pair kernel: a pair's odd whole tiles walk K downwards
    bool pair;             // CTA pairs: 256-row tiles, cta_group::2
    int max_pairs;         // co-resident clusters of 2 for the chosen pair kernel
    bool b_vnni_inkernel;  // blocked B re-laid inside the GEMM kernel
    bool b_repack;         // blocked B unpacked to row-major scratch first
    bool b_3d;             // B tensor map is the 3-D slab view
    bool b_kmajor;         // B is stored transposed, Bt[N][K]: K-major tiles by TMA, like A
    bool cluster_reduce;   // K splits of a tile = the CTAs of one cluster; partial sums meet in shared memory
    int tail_from, tail_splits;   // pair kernel: tiles >= tail_from (the last, partial wave) are shared out by k-blocks; -1: off.  tail_splits: the forced cut, else 0
    int sk_share, sk_max_segs;    // k-blocks of the tail per pair; partial slabs reserved per tail tile
    // SIMT
    int simt_tile;  // 128, 64 or 32
    int kt_per_split;
    int skinny_kc;  // FP32 skinny kernel: k per CTA
    // batch-reduce (normalised: batch >= 1, strides in elements)
    int batch;              // items reduced into one C (1 in a batched matmul)
    long long stride_a, stride_b;
    int gemms;              // independent GEMMs per run (batched matmul), else 1
    long long stride_c;
    // workspace layout
    size_t ws_repack_bytes, ws_partial_bytes;
    // device status word
    unsigned int* status_dev;
    // cached tensor maps
    CUtensorMap tmap_a, tmap_b, tmap_c;
    const void *cached_a, *cached_b, *cached_c;
    bool tma_store;        // row-major C without beta or K split: stored by TMA, 32 x 32 boxes
    nk::EncodeTiledFn encode;
    char name[128];
    char cuda_err[256];
    int launches;
    // FP32 operands on the tensor cores: A and B are split into three BF16 planes each (workspace) and
    // `inner`, a BF16 batch-reduce plan over six (A plane, B plane) pairs, multiplies the cross terms
    nk_gemm_s* inner;
    long long plane_a, plane_b;   // elements per plane
    // set on such an inner plan: FP32 bias with 16-bit operands; batch item -> (A item, B item)
    bool bias_f32, item_remap;
    uint32_t item_map_a, item_map_b;
    // nk_gemm_run_host on large problems: 8 row chunks x up to 4 column panels pipelined over two copy
    // streams (made on first use)
    nk_gemm_s* chunk_plan;
    bool chunk_tried;      // the chunk plan was asked for once already (and, if chunk_plan is null, refused)
    int chunk_rows, chunk_panels;
    cudaStream_t h2d_stream, d2h_stream;
    cudaEvent_t ev_start, ev_done, ev_up[12], ev_g[32];
};

namespace nk {

static void set_err(nk_gemm_s* p, const char* what, cudaError_t e) {
    snprintf(p->cuda_err, sizeof(p->cuda_err), "%s: %s", what, cudaGetErrorString(e));
}

struct DeviceGuard {
    int prev = -1;
    bool changed = false;
    cudaError_t err = cudaSuccess;
    explicit DeviceGuard(int dev) {
        err = cudaGetDevice(&prev);
        if (err == cudaSuccess && prev != dev) {
            err = cudaSetDevice(dev);
            changed = (err == cudaSuccess);
        }
    }
    ~DeviceGuard() {
        if (changed) cudaSetDevice(prev);
    }
};

static inline bool is16(int dt) { return dt == NK_BF16 || dt == NK_F16; }   // a 16-bit element type
static inline bool is_s8(const nk_gemm_desc_t& d) { return d.in_dtype == NK_S8; }
static inline bool is_f8(const nk_gemm_desc_t& d) { return d.in_dtype == NK_E4M3 || d.in_dtype == NK_E5M2; }
static inline bool is_8bit(const nk_gemm_desc_t& d) { return is_s8(d) || is_f8(d); }
// k elements in one stage row of the tensor-core kernels (128 bytes)
static inline int kblock(const nk_gemm_desc_t& d) { return is_8bit(d) ? 2 * UMMA_BK : UMMA_BK; }
static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int ceil_div(int64_t a, int64_t b) { return static_cast<int>((a + b - 1) / b); }

// tcgen05 instruction descriptor, kind::f16: D format FP32 (bit 4), A and B format at bits 7 and
// 10 (0 = FP16, 1 = BF16), B major-ness (bit 16: 0 = K-major, 1 = N-major), N/8 at bit 17,
// M/16 at bit 24.  A is always K-major.
static uint32_t make_idesc(int m, int n, bool b_n_major, bool f16, bool s8 = false, int f8_format = -1) {
    uint32_t d = 0;
    if (f8_format >= 0) {
        // kind::f8f6f4: D format FP32 (1 at bit 4), A and B format at bits 7 and 10 (0 = E4M3, 1 = E5M2)
        d |= 1u << 4;
        d |= static_cast<uint32_t>(f8_format) << 7;
        d |= static_cast<uint32_t>(f8_format) << 10;
        d |= static_cast<uint32_t>(n >> 3) << 17;
        d |= static_cast<uint32_t>(m >> 4) << 24;
        return d;   // both operands K-major
    }
    if (s8) {
        // kind::i8: D format INT32 (2 at bit 4), A and B format signed 8-bit (1 at bits 7 and 10)
        d |= 2u << 4;
        d |= 1u << 7;
        d |= 1u << 10;
        d |= static_cast<uint32_t>(n >> 3) << 17;
        d |= static_cast<uint32_t>(m >> 4) << 24;
        return d;   // both operands K-major
    }
    d |= 1u << 4;
    d |= (f16 ? 0u : 1u) << 7;
    d |= (f16 ? 0u : 1u) << 10;
    d |= (b_n_major ? 1u : 0u) << 16;
    d |= static_cast<uint32_t>(n >> 3) << 17;
    d |= static_cast<uint32_t>(m >> 4) << 24;
    return d;
}

// The same for the swapped-operand skinny kernel: the MMA's A operand is the GEMM's B tile (MN-major
// when B is row-major [K][N], bit 15; K-major when B is stored transposed), its B operand the GEMM's
// A tile (K-major), M = 128, N = the padded row count of the GEMM's A.
static uint32_t make_idesc_swap(int n, bool a_mn_major, bool f16) {
    uint32_t d = 0;
    d |= 1u << 4;
    d |= (f16 ? 0u : 1u) << 7;
    d |= (f16 ? 0u : 1u) << 10;
    d |= (a_mn_major ? 1u : 0u) << 15;
    d |= static_cast<uint32_t>(n >> 3) << 17;
    d |= static_cast<uint32_t>(UMMA_BM >> 4) << 24;
    return d;
}

template <typename K>
static cudaError_t allow_smem(K kernel, int bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

static int umma_stages_for(int bn) { return bn == 256 ? 4 : bn == 128 ? 6 : 8; }

// Plan-time choice of (single CTA | CTA pair) x tile N x K splits for the BF16 kernel: the
// counterpart of the paper's tile-size selection (Section 5a, found there by manual search).
// A small cost model, fitted to timings on B200, is evaluated for every candidate:
//   time = fixed + rounds * k-blocks-per-unit * t_kb(variant) [+ split-K partials and reduce],
// floored by the HBM time of the operands.  t_kb is nearly independent of the tile width
// (the stage pipeline is latency bound), so wide tiles win whenever they do not cost rounds.
struct UmmaChoice { bool pair; int bn; int splits; double us; };

static int desc_batch(const nk_gemm_desc_t& d) { return (d.batch > 1 && !d.batch_independent) ? static_cast<int>(d.batch) : 1; }
static int desc_gemms(const nk_gemm_desc_t& d) { return (d.batch > 1 && d.batch_independent) ? static_cast<int>(d.batch) : 1; }

// Co-resident clusters of the cluster split-K variant (pair?, tile N, VNNI?, splits), as the driver
// reports them for the current device; asked once per device and variant and remembered.
static int max_clusters_for(bool pair, int bn, bool vnni, int splits, int kind);

// K splits can meet inside a cluster (no partials in global memory, no second kernel) when there
// are 2, 4 or 8 of them (2 or 4 pairs) and all the units of the plan are resident at once (one
// unit per CTA; large clusters leave a few SMs of every GPC unused, which the driver's answer
// accounts for).
static bool cluster_reduce_fits(const nk_gemm_desc_t& d, int sms, bool pair, int bn, int eff_splits) {
    (void)sms;
    if (d.flags & NK_FLAG_SEPARATE_REDUCE) return false;
    if (eff_splits != 2 && eff_splits != 4 && !(eff_splits == 8 && !pair)) return false;
    const int64_t clusters = static_cast<int64_t>(desc_gemms(d)) * ceil_div(d.M, pair ? 2 * UMMA_BM : UMMA_BM) * ceil_div(d.N, bn);
    const bool vnni = d.layout_b == NK_BLOCKED32 && !(d.flags & NK_FLAG_REPACK_B);
    return clusters <= max_clusters_for(pair, bn, vnni, eff_splits, is_f8(d) ? 2 : is_s8(d) ? 1 : 0);
}

static double umma_model_us(const nk_gemm_desc_t& d, int sms, bool pair, int bn, int splits) {
    const int kb_total = desc_batch(d) * ceil_div(d.K, kblock(d));
    const int per = ceil_div(kb_total, splits);
    const int eff_splits = ceil_div(kb_total, per);
    const int64_t tiles = static_cast<int64_t>(desc_gemms(d)) * ceil_div(d.M, pair ? 256 : 128) * ceil_div(d.N, bn);
    const int64_t units = tiles * eff_splits;
    const int workers = pair ? sms / 2 : sms;
    const double rounds = static_cast<double>((units + workers - 1) / workers);
    // Fitted to kernel-only durations (one-pass ncu captures, cold L2) of every variant on the MLP
    // shapes.  A k-block costs 0.33-0.38 us whatever the tile (the SM's operand feed from L2, or
    // the MMA at N = 256), a little more when nearly every SM streams at once; start-up is
    // 5.4-7.3 us; the epilogue of the last tile is not hidden (0.35 us per 32 columns, 0.5 in a
    // pair: the SM's store path); a cluster reduction costs 1.2 us (barrier, receive wait) plus
    // 1.1 us per 32 x 32 piece a warp sends: the SM-to-SM path moves only ~13 KB per microsecond
    // per CTA, so two splits (half of the pieces stay at home) usually beat four.
    const bool busy = units > 100;
    double t_kb, start;  // microseconds per 64-wide k-block of one unit; start-up of the kernel
    if (pair) {
        t_kb = bn == 256 ? (rounds > 1 ? 0.385 : busy ? 0.34 : 0.325) : (busy ? 0.35 : 0.335);
        start = bn == 256 ? 7.3 : 6.4;
    } else {
        t_kb = bn == 256 ? (busy ? 0.42 : 0.37) : bn == 128 ? (busy ? 0.35 : 0.335) : 0.31;
        start = bn == 256 ? 6.0 : bn == 128 ? 5.4 : 5.5;
    }
    if (d.layout_b == NK_BLOCKED32 && !(d.flags & NK_FLAG_REPACK_B)) {
        // VNNI-blocked B is re-laid in place by four warps: the CTA's share of B crosses shared memory
        // four times instead of twice (TMA write, re-layout read and write, MMA read), and a k-block
        // then costs what the shared-memory port needs for all of a stage's traffic (~250 KB/us)
        const int cols = pair ? bn / 2 : bn;
        const double vnni = (32.0 + cols / 2.0) / 250.0;
        if (vnni > t_kb) t_kb = vnni;
    }
    const double eo = is16(d.out_dtype) ? 2.0 : 4.0;
    const double mn = static_cast<double>(d.M) * d.N;
    const double chunks = bn / 32.0;
    double us = start + rounds * per * t_kb;
    if (eff_splits > 1 && cluster_reduce_fits(d, sms, pair, bn, eff_splits)) {
        us += 1.2 + 1.1 * chunks * (eff_splits - 1) / eff_splits + (pair ? 0.5 : 0.0);
    } else {
        us += chunks * (pair ? 0.5 : 0.35);
        // two kernels: the reduce kernel, the gap before it, and the partials written and read back
        if (eff_splits > 1) us += 5.5 + eff_splits * mn * 4.0 / 3.0e6 + (eff_splits * 4.0 + eo) * mn / 5.0e6;
    }
    const double bytes = 2.0 * desc_batch(d) * (static_cast<double>(d.M) * d.K + static_cast<double>(d.K) * d.N) + eo * mn;
    const double hbm_us = bytes / 5.2e6;  // ~80 % of the copy bandwidth, bytes per microsecond
    return us > hbm_us ? us : hbm_us;
}

static void choose_umma(nk_gemm_s* p) {
    const nk_gemm_desc_t& d = p->d;
    const int sms = p->sm_count;
    const int kb_total = desc_batch(d) * ceil_div(d.K, kblock(d));
    const int forced_bn = (d.flags >> NK_FLAG_TILE_N_SHIFT) & 0xF;
    const int forced_s = (d.flags >> NK_FLAG_SPLITK_SHIFT) & 0xFF;
    const int split_cands[8] = {1, 2, 3, 4, 6, 8, 12, 16};
    UmmaChoice best = {false, 64, 1, 1e30};
    for (int pr = 0; pr < 2; ++pr) {
        const bool pair = pr == 1;
        if (pair && (d.flags & NK_FLAG_SINGLE_CTA)) continue;
        if (!pair && (d.flags & NK_FLAG_CTA_PAIR) && forced_bn != 2) continue;
        if (pair && d.M <= UMMA_BM && !(d.flags & NK_FLAG_CTA_PAIR)) continue;
        for (int bn = 64; bn <= 256; bn *= 2) {
            if (pair && bn == 64) continue;
            if (forced_bn >= 2 && forced_bn <= 4 && bn != (32 << (forced_bn - 1))) continue;
            for (int si = 0; si < 8; ++si) {
                int splits = forced_s > 0 ? forced_s : split_cands[si];
                if (forced_s > 0 && si > 0) break;
                if (splits > kb_total) splits = kb_total;
                if (forced_s == 0 && splits > 1) {
                    if (kb_total / splits < 4) continue;  // >= 4 k-blocks per split
                    if (static_cast<double>(splits) * desc_gemms(d) * d.M * d.N * 4.0 > 256.0 * 1024 * 1024) continue;
                }
                const double us = umma_model_us(d, sms, pair, bn, splits);
                if (us < best.us) best = {pair, bn, splits, us};
            }
        }
    }
    if (best.us >= 1e30) best = {false, 64, forced_s > 0 ? forced_s : 1, 0.0};  // contradictory overrides
    int splits = best.splits;
    if (splits > kb_total) splits = kb_total;
    if (splits < 1) splits = 1;
    const int per = ceil_div(kb_total, splits);
    splits = ceil_div(kb_total, per);  // no empty split
    p->pair = best.pair;
    p->bn = best.bn;
    p->stages = best.pair ? (best.bn == 256 ? 6 : 8) : umma_stages_for(best.bn);
    p->splits = splits;
    p->group_m = 8;
    p->serpentine = false;
    {
        // tuning override of the raster: bits 28-30 pick the group size (7: no K serpentine), bit 31 switches the serpentine sweep off
        static const int kGroups[8] = {8, 4, 6, 12, 16, 24, 2, 8};
        p->group_m = kGroups[(d.flags >> NK_FLAG_RASTER_SHIFT) & 7u];
        p->k_serpentine = ((d.flags >> NK_FLAG_RASTER_SHIFT) & 7u) != 7u;   // code 7: K always upwards
        p->serpentine = ((d.flags >> (NK_FLAG_RASTER_SHIFT + 3)) & 1u) == 0;
    }
    p->cluster_reduce = splits > 1 && cluster_reduce_fits(d, sms, best.pair, best.bn, splits);
}

// Plan-time choice of tile and K splits for the FP32 kernel (the counterpart of the paper's
// register-tile selection, Section 5a).  Model, fitted to B200 timings: an SM holds `res`
// CTAs of a variant; a CTA's 16-wide k-tile costs tile^2 * 16 FMAs on 128 lanes, slowed by
// the CTAs sharing the SM and by the variant's efficiency (wide thread tiles need fewer
// shared-memory loads per FMA); units are scheduled in waves of sms * res.
static double simt_model_us(const nk_gemm_desc_t& d, int sms, int tile, int splits) {
    const int ktiles = desc_batch(d) * ceil_div(d.K, SIMT_BK);
    const int per = ceil_div(ktiles, splits);
    const int eff_splits = ceil_div(ktiles, per);
    const int64_t tiles = static_cast<int64_t>(desc_gemms(d)) * ceil_div(d.M, tile) * ceil_div(d.N, tile);
    const int64_t units = tiles * eff_splits;
    const int res = tile == 128 ? 2 : tile == 64 ? 4 : 16;
    const double eff = tile == 128 ? ((d.flags & NK_FLAG_SCALAR_FMA) ? 0.68 : 0.82) : tile == 64 ? 0.50 : 0.37;
    const int64_t slots = static_cast<int64_t>(sms) * res;
    const int64_t full_waves = units / slots;
    const int64_t rest = units - full_waves * slots;
    const double clk_per_kt = static_cast<double>(tile) * tile * SIMT_BK / 128.0;   // one CTA alone on an SM
    const double us_per_kt = clk_per_kt / 1965.0 / eff;
    // a CTA prefetches one k-tile only, so a k-tile never takes less than a global-load round trip
    const double lat_us = 0.85;
    auto kt_us = [&](double sharing) { const double t = us_per_kt * sharing; return t > lat_us ? t : lat_us; };
    double us = 8.0 + full_waves * per * kt_us(res);
    if (rest > 0) us += per * kt_us(static_cast<double>((rest + sms - 1) / sms));
    const double mn = static_cast<double>(d.M) * d.N;
    if (eff_splits > 1) us += 3.0 + (2.0 * eff_splits + 1.0) * mn * 4.0 / 4.0e6;
    const double bytes = 4.0 * (desc_batch(d) * (static_cast<double>(d.M) * d.K + static_cast<double>(d.K) * d.N) + mn);
    // small tiles keep few bytes in flight: they reach a fraction of the HBM bandwidth only
    const double hbm_us = bytes / (tile == 128 ? 5.0e6 : tile == 64 ? 3.5e6 : 1.8e6);
    return us > hbm_us ? us : hbm_us;
}

static void choose_simt(nk_gemm_s* p) {
    const nk_gemm_desc_t& d = p->d;
    const int sms = p->sm_count;
    const int ktiles = desc_batch(d) * ceil_div(d.K, SIMT_BK);
    const int forced = (d.flags >> NK_FLAG_TILE_N_SHIFT) & 0xF;
    const int forced_s = (d.flags >> NK_FLAG_SPLITK_SHIFT) & 0xFF;
    const int split_cands[10] = {1, 2, 3, 4, 6, 8, 12, 16, 24, 32};
    int best_tile = 32, best_splits = 1;
    double best_us = 1e30;
    for (int tile = 32; tile <= 128; tile *= 2) {
        if (forced >= 1 && forced <= 3 && tile != (16 << forced)) continue;
        for (int si = 0; si < 10; ++si) {
            int splits = forced_s > 0 ? forced_s : split_cands[si];
            if (forced_s > 0 && si > 0) break;
            if (splits > ktiles) splits = ktiles;
            if (forced_s == 0 && splits > 1) {
                if (ktiles / splits < 8) continue;   // >= 8 k-tiles (128 k) per split
                if (static_cast<double>(splits) * desc_gemms(d) * d.M * d.N * 4.0 > 256.0 * 1024 * 1024) continue;
            }
            const double us = simt_model_us(d, sms, tile, splits);
            if (us < best_us) { best_us = us; best_tile = tile; best_splits = splits; }
        }
    }
    int splits = best_splits;
    if (splits > ktiles) splits = ktiles;
    if (splits < 1) splits = 1;
    const int per = ceil_div(ktiles, splits);
    splits = ceil_div(ktiles, per);
    p->simt_tile = best_tile;
    p->splits = splits;
    p->kt_per_split = per;
}

// FP32, M <= 32: the streaming kernel.  K is cut so that about four CTAs per SM stream B at
// once; a CTA's slice of A (rows x k-chunk) must fit its 32 KB of shared memory.
static void choose_skinny(nk_gemm_s* p) {
    const nk_gemm_desc_t& d = p->d;
    const int mr = d.M <= 16 ? 16 : 32;
    const int kc_max = SKINNY_A_FLOATS / mr;
    const int col_tiles = ceil_div(d.N, SKINNY_COLS);
    const int forced_s = (d.flags >> NK_FLAG_SPLITK_SHIFT) & 0xFF;
    int want = forced_s > 0 ? forced_s : ceil_div(4 * p->sm_count, col_tiles);
    if (want < 1) want = 1;
    int kc = ceil_div(ceil_div(d.K, want), 8) * 8;
    if (kc < 64 && forced_s == 0) kc = 64;
    if (kc > kc_max) kc = kc_max;
    if (kc > ceil_div(d.K, 8) * 8) kc = ceil_div(d.K, 8) * 8;
    p->skinny_kc = kc;
    p->splits = ceil_div(d.K, kc);
}

static nk_status_t encode_maps(nk_gemm_s* p, const void* A, const void* B) {
    if (p->cached_a == A && p->cached_b == B) return NK_OK;
    const nk_gemm_desc_t& d = p->d;
    const CUtensorMapDataType half_type = is_8bit(d) ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                          : d.in_dtype == NK_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const cuuint64_t esz = is_8bit(d) ? 1 : 2;   // bytes per operand element
    CUresult r;
    if (d.layout_a == NK_BLOCKED32) {
        // [M/32][K/32][32][32] as a 4-D tensor (k, m, k-block, m-block): a box of
        // 32 x 32 x 1 x 4 lands in shared memory as 128 rows of 32 consecutive k (64 B).
        // Batch items (stride_a elements apart) are the fifth dimension.
        cuuint64_t dims[5] = {32, 32, static_cast<cuuint64_t>(d.K / 32), static_cast<cuuint64_t>(d.M / 32),
                              static_cast<cuuint64_t>(p->batch * p->gemms)};
        cuuint64_t strides[4] = {32 * 2, 1024 * 2, static_cast<cuuint64_t>(d.K / 32) * 1024 * 2,
                                 static_cast<cuuint64_t>(p->stride_a) * 2};
        cuuint32_t box[5] = {32, 32, 1, 4, 1};
        cuuint32_t es[5] = {1, 1, 1, 1, 1};
        r = p->encode(&p->tmap_a, half_type, 5, const_cast<void*>(A), dims, strides,
                      box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        // A row-major [batch][M][K] (batch items stride_a elements apart): (k, m, item)
        cuuint64_t dims[3] = {static_cast<cuuint64_t>(d.K), static_cast<cuuint64_t>(d.M),
                              static_cast<cuuint64_t>(p->batch * p->gemms)};
        cuuint64_t strides[2] = {static_cast<cuuint64_t>(d.K) * esz, static_cast<cuuint64_t>(p->stride_a) * esz};
        cuuint32_t box[3] = {static_cast<cuuint32_t>(kblock(d)), static_cast<cuuint32_t>(p->variant == V_SWAP ? p->swap_mp : UMMA_BM), 1};   // 128 bytes of k per row
        cuuint32_t es[3] = {1, 1, 1};
        r = p->encode(&p->tmap_a, half_type, 3, const_cast<void*>(A), dims, strides,
                      box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) {
        snprintf(p->cuda_err, sizeof(p->cuda_err), "cuTensorMapEncodeTiled(A) failed: %d", (int)r);
        return NK_ERR_CUDA;
    }
    if (p->b_kmajor) {
        // B stored transposed, Bt[batch][N][K] (K contiguous): (k, n, item), one box of 128 bytes of k by
        // the columns a CTA covers, K-major in shared memory exactly like A's tile
        const int cols = p->variant == V_SWAP ? 128 : p->pair ? p->bn / 2 : p->bn;
        cuuint64_t dims[3] = {static_cast<cuuint64_t>(d.K), static_cast<cuuint64_t>(d.N),
                              static_cast<cuuint64_t>(p->batch * p->gemms)};
        cuuint64_t strides[2] = {static_cast<cuuint64_t>(d.K) * esz, static_cast<cuuint64_t>(p->stride_b) * esz};
        cuuint32_t box[3] = {static_cast<cuuint32_t>(kblock(d)), static_cast<cuuint32_t>(cols), 1};
        cuuint32_t es[3] = {1, 1, 1};
        r = p->encode(&p->tmap_b, half_type, 3, const_cast<void*>(B), dims, strides,
                      box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            snprintf(p->cuda_err, sizeof(p->cuda_err), "cuTensorMapEncodeTiled(B transposed) failed: %d", (int)r);
            return NK_ERR_CUDA;
        }
    } else if (!p->b_vnni_inkernel) {
        // B row-major [K][N], N contiguous.  When N is a multiple of 64 the map is the 3-D view
        // (n within a 64-column slab, k, slab): one box brings all the slabs of a stage, each
        // as 64 k-rows of 128 B.  Otherwise 64 (n) x 64 (k) boxes, one per slab.
        p->b_3d = d.N % 64 == 0;
        const int slabs = p->variant == V_SWAP ? 2 : (p->pair ? p->bn / 2 : p->bn) / 64;
        if (p->b_3d) {
            // (n within slab, k, slab, item)
            cuuint64_t dims[4] = {64, static_cast<cuuint64_t>(d.K), static_cast<cuuint64_t>(d.N / 64),
                                  static_cast<cuuint64_t>(p->batch * p->gemms)};
            cuuint64_t strides[3] = {static_cast<cuuint64_t>(d.N) * 2, 128, static_cast<cuuint64_t>(p->stride_b) * 2};
            cuuint32_t box[4] = {64, UMMA_BK, static_cast<cuuint32_t>(slabs), 1};
            cuuint32_t es[4] = {1, 1, 1, 1};
            r = p->encode(&p->tmap_b, half_type, 4, const_cast<void*>(B), dims, strides,
                          box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) p->b_3d = false;   // fall back to per-slab boxes
        }
        if (!p->b_3d) {
            // (n, k, item)
            cuuint64_t dims[3] = {static_cast<cuuint64_t>(d.N), static_cast<cuuint64_t>(d.K),
                                  static_cast<cuuint64_t>(p->batch * p->gemms)};
            cuuint64_t strides[2] = {static_cast<cuuint64_t>(d.N) * 2, static_cast<cuuint64_t>(p->stride_b) * 2};
            cuuint32_t box[3] = {64, UMMA_BK, 1};
            cuuint32_t es[3] = {1, 1, 1};
            r = p->encode(&p->tmap_b, half_type, 3, const_cast<void*>(B), dims, strides,
                          box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        }
        if (r != CUDA_SUCCESS) {
            snprintf(p->cuda_err, sizeof(p->cuda_err), "cuTensorMapEncodeTiled(B) failed: %d", (int)r);
            return NK_ERR_CUDA;
        }
    } else {
        // B VNNI-blocked [N/32][K/32][16][32][2]: a k-pair row of a block is 64 elements (128 B), the
        // 16 rows of a block and the K/32 blocks of a column block follow one another, so the
        // operand is the 3-D tensor (64, K/2, N/32).  One box brings the 32 pair rows of a 64-deep
        // stage for all the column blocks a CTA covers, swizzled per 128-byte row; rows beyond
        // K/2 and column blocks beyond N/32 arrive as zeros.
        // INT8: the same bytes with four k per group: [N/32][K/32][8][32][4] is (128 elements, K/4, N/32).
        const int cols = p->pair ? p->bn / 2 : p->bn;
        const cuuint64_t group = 4 / esz;   // k per 32-bit word: 2 (16-bit) or 4 (8-bit)
        // Batch items (stride_b elements apart) are the fourth dimension.
        cuuint64_t dims[4] = {128 / esz, static_cast<cuuint64_t>(d.K) / group, static_cast<cuuint64_t>(d.N / 32),
                              static_cast<cuuint64_t>(p->batch * p->gemms)};
        cuuint64_t strides[3] = {128, static_cast<cuuint64_t>(d.K) * 32 * esz, static_cast<cuuint64_t>(p->stride_b) * esz};
        cuuint32_t box[4] = {static_cast<cuuint32_t>(128 / esz), UMMA_BK / 2, static_cast<cuuint32_t>(cols / 32), 1};
        cuuint32_t es[4] = {1, 1, 1, 1};
        r = p->encode(&p->tmap_b, half_type, 4, const_cast<void*>(B), dims, strides,
                      box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            snprintf(p->cuda_err, sizeof(p->cuda_err), "cuTensorMapEncodeTiled(B blocked) failed: %d", (int)r);
            return NK_ERR_CUDA;
        }
    }
    p->cached_a = A;
    p->cached_b = B;
    return NK_OK;
}

// C row-major [gemms][M][N] as (n, m, gemm): the epilogue stores 32 x 32 boxes from a swizzled
// staging tile; the TMA unit drops whatever lies beyond M or N.
static nk_status_t encode_c_map(nk_gemm_s* p, void* C) {
    if (!p->tma_store || p->cached_c == C) return NK_OK;
    const nk_gemm_desc_t& d = p->d;
    const bool bf16 = is16(d.out_dtype);
    const cuuint64_t es_bytes = bf16 ? 2 : 4;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(d.N), static_cast<cuuint64_t>(d.M), static_cast<cuuint64_t>(p->gemms)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(d.N) * es_bytes, static_cast<cuuint64_t>(p->stride_c) * es_bytes};
    cuuint32_t box[3] = {32, 32, 1};
    cuuint32_t es[3] = {1, 1, 1};
    // a box row is 128 bytes of FP32 (128-byte swizzle) or 64 bytes of BF16 (64-byte swizzle)
    CUresult r = p->encode(&p->tmap_c, d.out_dtype == NK_S32 ? CU_TENSOR_MAP_DATA_TYPE_INT32 : !bf16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : d.out_dtype == NK_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, C,
                           dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(p->cuda_err, sizeof(p->cuda_err), "cuTensorMapEncodeTiled(C) failed: %d", (int)r);
        return NK_ERR_CUDA;
    }
    p->cached_c = C;
    return NK_OK;
}

template <int BN, int STAGES, bool VNNI, int KIND = 0>
static cudaError_t launch_umma_t(nk_gemm_s* p, const UmmaParams& up, int grid, cudaStream_t st) {
    umma_bf16_kernel<BN, STAGES, VNNI, false, KIND><<<grid, UMMA_THREADS, umma_smem_bytes(BN, STAGES), st>>>(
        p->tmap_a, p->tmap_b, p->tmap_c, up);
    return cudaGetLastError();
}

static cudaError_t launch_umma(nk_gemm_s* p, const UmmaParams& up, int grid, cudaStream_t st) {
    const bool v = p->b_vnni_inkernel;
    if (is_s8(p->d)) {   // 8-bit operands: B blocked and re-laid in the kernel, or stored transposed
        switch (p->bn) {
            case 256: return v ? launch_umma_t<256, 4, true, 1>(p, up, grid, st) : launch_umma_t<256, 4, false, 1>(p, up, grid, st);
            case 128: return v ? launch_umma_t<128, 6, true, 1>(p, up, grid, st) : launch_umma_t<128, 6, false, 1>(p, up, grid, st);
            default:  return v ? launch_umma_t<64, 8, true, 1>(p, up, grid, st) : launch_umma_t<64, 8, false, 1>(p, up, grid, st);
        }
    }
    if (is_f8(p->d)) {
        switch (p->bn) {
            case 256: return v ? launch_umma_t<256, 4, true, 2>(p, up, grid, st) : launch_umma_t<256, 4, false, 2>(p, up, grid, st);
            case 128: return v ? launch_umma_t<128, 6, true, 2>(p, up, grid, st) : launch_umma_t<128, 6, false, 2>(p, up, grid, st);
            default:  return v ? launch_umma_t<64, 8, true, 2>(p, up, grid, st) : launch_umma_t<64, 8, false, 2>(p, up, grid, st);
        }
    }
    switch (p->bn) {
        case 256: return v ? launch_umma_t<256, 4, true>(p, up, grid, st) : launch_umma_t<256, 4, false>(p, up, grid, st);
        case 128: return v ? launch_umma_t<128, 6, true>(p, up, grid, st) : launch_umma_t<128, 6, false>(p, up, grid, st);
        default:  return v ? launch_umma_t<64, 8, true>(p, up, grid, st) : launch_umma_t<64, 8, false>(p, up, grid, st);
    }
}

// Cluster split-K variants of both kernels: the cluster is `splits` CTAs (or pairs) wide and the
// grid is exactly the units; with `max_clusters` set only the occupancy of one cluster is queried.
template <typename Kernel>
static cudaError_t launch_clustered(Kernel kernel, nk_gemm_s* p, const UmmaParams& up, int ctas, int cluster, int threads,
                                    int smem, cudaStream_t st, int* max_clusters) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(max_clusters ? cluster : ctas));
    cfg.blockDim = dim3(static_cast<unsigned>(threads));
    cfg.dynamicSmemBytes = static_cast<size_t>(smem);
    cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = static_cast<unsigned>(cluster);
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (max_clusters) return cudaOccupancyMaxActiveClusters(max_clusters, kernel, &cfg);
    return cudaLaunchKernelEx(&cfg, kernel, p->tmap_a, p->tmap_b, p->tmap_c, up);
}

// `units` = tiles x splits; the single-CTA kernel runs one CTA per unit, the pair kernel two.
// KIND as in the kernels (0 = 16-bit floating point, 1 = INT8, 2 = 8-bit floating point).
template <int KIND>
static cudaError_t launch_cluster_k(nk_gemm_s* p, const UmmaParams& up, int units, int splits, cudaStream_t st,
                                    int* max_clusters) {
    const bool v = p->b_vnni_inkernel;
    const int th = UMMA_THREADS;
#define NK_CL(K, ctas, cl, smem) launch_clustered(K, p, up, ctas, cl, th, smem, st, max_clusters)
    if (p->pair) {
        if (p->bn == 256)
            return v ? NK_CL((umma_bf16_pair_kernel<256, 6, true, true, KIND>), 2 * units, 2 * splits, pair_smem_bytes(256, 6))
                     : NK_CL((umma_bf16_pair_kernel<256, 6, false, true, KIND>), 2 * units, 2 * splits, pair_smem_bytes(256, 6));
        return v ? NK_CL((umma_bf16_pair_kernel<128, 8, true, true, KIND>), 2 * units, 2 * splits, pair_smem_bytes(128, 8))
                 : NK_CL((umma_bf16_pair_kernel<128, 8, false, true, KIND>), 2 * units, 2 * splits, pair_smem_bytes(128, 8));
    }
    if (p->bn == 256)
        return v ? NK_CL((umma_bf16_kernel<256, 4, true, true, KIND>), units, splits, umma_smem_bytes(256, 4))
                 : NK_CL((umma_bf16_kernel<256, 4, false, true, KIND>), units, splits, umma_smem_bytes(256, 4));
    if (p->bn == 128)
        return v ? NK_CL((umma_bf16_kernel<128, 6, true, true, KIND>), units, splits, umma_smem_bytes(128, 6))
                 : NK_CL((umma_bf16_kernel<128, 6, false, true, KIND>), units, splits, umma_smem_bytes(128, 6));
    return v ? NK_CL((umma_bf16_kernel<64, 8, true, true, KIND>), units, splits, umma_smem_bytes(64, 8))
             : NK_CL((umma_bf16_kernel<64, 8, false, true, KIND>), units, splits, umma_smem_bytes(64, 8));
#undef NK_CL
}

static cudaError_t launch_cluster(nk_gemm_s* p, const UmmaParams& up, int units, int splits, cudaStream_t st,
                                  int* max_clusters) {
    return is_f8(p->d) ? launch_cluster_k<2>(p, up, units, splits, st, max_clusters)
           : is_s8(p->d) ? launch_cluster_k<1>(p, up, units, splits, st, max_clusters)
                         : launch_cluster_k<0>(p, up, units, splits, st, max_clusters);
}

static int max_clusters_for(bool pair, int bn, bool vnni, int splits, int kind) {
    static std::mutex mu;
    static int cache[16][3][2][3][2][9];   // [device][kind][pair?][tile][VNNI?][splits]: 0 = not asked yet, -1 = none
    const int bi = bn == 256 ? 2 : bn == 128 ? 1 : 0;
    if (splits < 2 || splits > 8) return 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 0; }
    nk_gemm_s tmp;
    memset(&tmp, 0, sizeof(tmp));
    tmp.pair = pair;
    tmp.bn = bn;
    tmp.b_vnni_inkernel = vnni;
    tmp.d.in_dtype = kind == 2 ? NK_E4M3 : kind == 1 ? NK_S8 : NK_BF16;
    auto ask = [&]() {
        int n = 0;
        if (launch_cluster(&tmp, UmmaParams(), 0, splits, nullptr, &n) != cudaSuccess || n <= 0) {
            cudaGetLastError();
            n = -1;
        }
        return n;
    };
    if (dev < 0 || dev >= 16) { const int n = ask(); return n > 0 ? n : 0; }   // beyond the cache: ask every time
    std::lock_guard<std::mutex> lock(mu);
    int& c = cache[dev][kind][pair ? 1 : 0][bi][vnni ? 1 : 0][splits];
    if (c == 0) c = ask();
    return c > 0 ? c : 0;
}

template <int BN, int STAGES, bool VNNI, int KIND = 0>
static cudaError_t launch_pair_t(nk_gemm_s* p, const UmmaParams& up, int pairs, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(2 * pairs));
    cfg.blockDim = dim3(UMMA_THREADS);
    cfg.dynamicSmemBytes = pair_smem_bytes(BN, STAGES);
    cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, umma_bf16_pair_kernel<BN, STAGES, VNNI, false, KIND>, p->tmap_a, p->tmap_b, p->tmap_c, up);
}

static cudaError_t launch_pair(nk_gemm_s* p, const UmmaParams& up, int pairs, cudaStream_t st) {
    const bool v = p->b_vnni_inkernel;
    if (is_s8(p->d)) {
        if (p->bn == 256) return v ? launch_pair_t<256, 6, true, 1>(p, up, pairs, st) : launch_pair_t<256, 6, false, 1>(p, up, pairs, st);
        return v ? launch_pair_t<128, 8, true, 1>(p, up, pairs, st) : launch_pair_t<128, 8, false, 1>(p, up, pairs, st);
    }
    if (is_f8(p->d)) {
        if (p->bn == 256) return v ? launch_pair_t<256, 6, true, 2>(p, up, pairs, st) : launch_pair_t<256, 6, false, 2>(p, up, pairs, st);
        return v ? launch_pair_t<128, 8, true, 2>(p, up, pairs, st) : launch_pair_t<128, 8, false, 2>(p, up, pairs, st);
    }
    if (p->bn == 256) return v ? launch_pair_t<256, 6, true>(p, up, pairs, st) : launch_pair_t<256, 6, false>(p, up, pairs, st);
    return v ? launch_pair_t<128, 8, true>(p, up, pairs, st) : launch_pair_t<128, 8, false>(p, up, pairs, st);
}

template <int BN, int STAGES, bool VNNI>
static cudaError_t pair_occupancy(int* out) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2);
    cfg.blockDim = dim3(UMMA_THREADS);
    cfg.dynamicSmemBytes = pair_smem_bytes(BN, STAGES);
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaOccupancyMaxActiveClusters(out, umma_bf16_pair_kernel<BN, STAGES, VNNI>, &cfg);
}

static cudaError_t prepare_simt_attrs() {
    return allow_smem(simt_f32_async_kernel<128, 128, 8, 16, true>, simt_async_smem_bytes<128, 128>());
}

// Every tensor-core kernel instantiation needs more dynamic shared memory than the default limit
// allows.  The attribute is per device: the table below is walked once for each device that
// creates a plan, not on every nk_gemm_create.
template <int BN, int ST, bool V, bool CL, int KIND>
static cudaError_t attr_single() { return allow_smem(umma_bf16_kernel<BN, ST, V, CL, KIND>, umma_smem_bytes(BN, ST)); }
template <int BN, int ST, bool V, bool CL, int KIND>
static cudaError_t attr_pair() { return allow_smem(umma_bf16_pair_kernel<BN, ST, V, CL, KIND>, pair_smem_bytes(BN, ST)); }

typedef cudaError_t (*AttrFn)();
#define NK_ATTR_VARIANTS(FN, BN, ST, KIND, CL) FN<BN, ST, false, CL, KIND>, FN<BN, ST, true, CL, KIND>
#define NK_ATTR_TILES(KIND, CL)                                                                      \
    NK_ATTR_VARIANTS(attr_single, 256, 4, KIND, CL), NK_ATTR_VARIANTS(attr_single, 128, 6, KIND, CL), \
    NK_ATTR_VARIANTS(attr_single, 64, 8, KIND, CL), NK_ATTR_VARIANTS(attr_pair, 256, 6, KIND, CL),    \
    NK_ATTR_VARIANTS(attr_pair, 128, 8, KIND, CL)
static const AttrFn kUmmaAttrTable[] = {
    NK_ATTR_TILES(0, false), NK_ATTR_TILES(0, true),   // 16-bit floating point, plain and cluster split-K
    NK_ATTR_TILES(1, false), NK_ATTR_TILES(1, true),   // INT8
    NK_ATTR_TILES(2, false), NK_ATTR_TILES(2, true),   // 8-bit floating point
};
#undef NK_ATTR_TILES
#undef NK_ATTR_VARIANTS

static cudaError_t prepare_umma_attrs(int device) {
    static std::mutex mu;
    static bool done[64];
    std::lock_guard<std::mutex> lock(mu);
    if (device >= 0 && device < 64 && done[device]) return cudaSuccess;
    for (const AttrFn fn : kUmmaAttrTable) {
        const cudaError_t e = fn();
        if (e != cudaSuccess) return e;
    }
    if (device >= 0 && device < 64) done[device] = true;
    return cudaSuccess;
}

static cudaError_t launch_simt(nk_gemm_s* p, const SimtParams& sp, cudaStream_t st) {
    const int t = p->simt_tile;
    dim3 grid(ceil_div(sp.N, t), ceil_div(sp.M, t), sp.splits * sp.gemms);
    // 128-tile: 128 threads with 8 x 16 thread tiles and packed FMAs (or, on request, the 256-thread
    // scalar-FFMA kernel with a register-staged double buffer); all through a three-stage cp.async
    // pipeline except the scalar one.
    if (t == 128 && (p->d.flags & NK_FLAG_SCALAR_FMA)) simt_f32_kernel<128, 128, 8, 8><<<grid, 256, 0, st>>>(sp);
    else if (t == 128) simt_f32_async_kernel<128, 128, 8, 16, true><<<grid, 128, simt_async_smem_bytes<128, 128>(), st>>>(sp);
    else if (t == 64) simt_f32_async_kernel<64, 64, 4, 4, false><<<grid, 256, simt_async_smem_bytes<64, 64>(), st>>>(sp);
    else simt_f32_async_kernel<32, 32, 4, 4, false><<<grid, 64, simt_async_smem_bytes<32, 32>(), st>>>(sp);
    return cudaGetLastError();
}

}  // namespace nk

using namespace nk;

extern "C" {

const char* nk_status_str(nk_status_t s) {
    switch (s) {
        case NK_OK: return "ok";
        case NK_ERR_INVALID_ARG: return "invalid argument";
        case NK_ERR_UNSUPPORTED: return "unsupported configuration";
        case NK_ERR_MISALIGNED: return "misaligned pointer or size";
        case NK_ERR_WORKSPACE: return "workspace missing or too small";
        case NK_ERR_DEVICE: return "no usable sm_100 CUDA device";
        case NK_ERR_CUDA: return "CUDA call failed";
        case NK_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

nk_status_t nk_gemm_create(const nk_gemm_desc_t* desc, nk_gemm_t* out) {
    if (out) *out = nullptr;
    if (!desc || !out) return NK_ERR_INVALID_ARG;
    const nk_gemm_desc_t& d = *desc;
    if (d.M <= 0 || d.N <= 0 || d.K <= 0) return NK_ERR_INVALID_ARG;
    if (d.M > (1 << 24) || d.N > (1 << 24) || d.K > (1 << 24)) return NK_ERR_UNSUPPORTED;
    if (d.M * d.N >= (1ll << 31) || d.M * d.K >= (1ll << 33) || d.K * d.N >= (1ll << 33)) return NK_ERR_UNSUPPORTED;
    if (d.in_dtype != NK_F32 && !is16(d.in_dtype) && !is_8bit(d)) return NK_ERR_INVALID_ARG;
    if (d.out_dtype != NK_F32 && !is16(d.out_dtype) && d.out_dtype != NK_S32) return NK_ERR_INVALID_ARG;
    if (d.out_dtype == NK_S32 && d.in_dtype != NK_S8) return NK_ERR_INVALID_ARG;   // an INT32 C belongs to INT8 operands
    if (is_f8(d)) {
        // 8-bit floating-point operands: A row-major, B packed in groups of four inside 32 x 32 blocks, FP32 C
        if (d.out_dtype != NK_F32) return NK_ERR_INVALID_ARG;
        if (d.layout_a != NK_ROW_MAJOR || d.layout_b == NK_ROW_MAJOR || d.layout_c != NK_ROW_MAJOR) return NK_ERR_UNSUPPORTED;
        if (d.batch > 1) return NK_ERR_UNSUPPORTED;
        if (d.flags & NK_FLAG_REPACK_B) return NK_ERR_UNSUPPORTED;
        const uint32_t fk = d.flags & NK_FLAG_KERNEL_MASK;
        if (fk == NK_FLAG_KERNEL_NAIVE || fk == NK_FLAG_KERNEL_SIMT) return NK_ERR_UNSUPPORTED;
    }
    if (d.in_dtype == NK_S8) {
        // the Int8 dot product: A row-major, B packed in groups of four inside 32 x 32 blocks; C is the exact
        // INT32 sum, or FP32 = scale * sum with the epilogue (quantised layer)
        if (d.out_dtype != NK_S32 && d.out_dtype != NK_F32) return NK_ERR_INVALID_ARG;
        if (d.layout_a != NK_ROW_MAJOR || d.layout_b == NK_ROW_MAJOR || d.layout_c != NK_ROW_MAJOR) return NK_ERR_UNSUPPORTED;
        if (d.beta != 0 || d.batch > 1) return NK_ERR_UNSUPPORTED;
        if (d.out_dtype == NK_S32 && d.epilogue != NK_EPI_NONE) return NK_ERR_UNSUPPORTED;
        if (d.out_dtype == NK_F32 && !(std::isfinite(d.scale) && d.scale != 0.0f)) return NK_ERR_INVALID_ARG;
        if (d.flags & NK_FLAG_REPACK_B) return NK_ERR_UNSUPPORTED;
        const uint32_t fk = d.flags & NK_FLAG_KERNEL_MASK;
        if (fk == NK_FLAG_KERNEL_NAIVE || fk == NK_FLAG_KERNEL_SIMT) return NK_ERR_UNSUPPORTED;
        if (d.K >= (1ll << 17)) return NK_ERR_UNSUPPORTED;   // INT32 accumulation is exact below 2^17 terms
    }
    if (d.layout_a != NK_ROW_MAJOR && d.layout_a != NK_BLOCKED32) return NK_ERR_INVALID_ARG;
    if (d.layout_b != NK_ROW_MAJOR && d.layout_b != NK_BLOCKED32 && d.layout_b != NK_TRANSPOSED) return NK_ERR_INVALID_ARG;
    if (d.layout_b == NK_TRANSPOSED) {
        // Bt[N][K]: 16-bit and 8-bit operands (the tensor-core kernels); rows of K elements must be 16-byte multiples
        if (d.in_dtype == NK_F32) return NK_ERR_UNSUPPORTED;
        if ((d.flags & NK_FLAG_KERNEL_MASK) == NK_FLAG_KERNEL_NAIVE || (d.flags & NK_FLAG_REPACK_B)) return NK_ERR_UNSUPPORTED;
        if (d.K % 16 || d.N % 8) return NK_ERR_MISALIGNED;
    }
    if (d.epilogue != NK_EPI_NONE && d.epilogue != NK_EPI_BIAS_RELU) return NK_ERR_INVALID_ARG;
    if (is16(d.out_dtype) && d.in_dtype != d.out_dtype) return NK_ERR_INVALID_ARG;   // a 16-bit C has the operands' type
    const bool blocked = d.layout_a == NK_BLOCKED32 || d.layout_b == NK_BLOCKED32;
    if (blocked && !is16(d.in_dtype) && !is_8bit(d)) return NK_ERR_UNSUPPORTED;
    if (d.layout_a == NK_BLOCKED32 && (d.M % 32 || d.K % 32)) return NK_ERR_MISALIGNED;
    if (d.layout_b == NK_BLOCKED32 && (d.N % 32 || d.K % 32)) return NK_ERR_MISALIGNED;
    if (d.beta != 0 && d.beta != 1) return NK_ERR_INVALID_ARG;
    if (d.batch < 0 || d.stride_a < 0 || d.stride_b < 0) return NK_ERR_INVALID_ARG;
    const int64_t nbatch = d.batch > 1 ? d.batch : 1;
    const int64_t str_a = d.stride_a > 0 ? d.stride_a : d.M * d.K;
    const int64_t str_b = d.stride_b > 0 ? d.stride_b : d.K * d.N;
    if (nbatch > 1) {
        if (nbatch > 65535 || nbatch * d.K >= (1ll << 24)) return NK_ERR_UNSUPPORTED;
        const int64_t gran = is16(d.in_dtype) ? 8 : 4;
        if (str_a % gran || str_b % gran) return NK_ERR_MISALIGNED;
        if (str_a < d.M * d.K || str_b < d.K * d.N) return NK_ERR_INVALID_ARG;   // items must not overlap
    }
    if (d.layout_c != NK_ROW_MAJOR && d.layout_c != NK_BLOCKED32) return NK_ERR_INVALID_ARG;
    if (d.layout_c == NK_BLOCKED32) {
        if (!is16(d.in_dtype)) return NK_ERR_UNSUPPORTED;
        if (d.M % 32 || d.N % 32) return NK_ERR_MISALIGNED;
    }
    if (d.batch_independent != 0 && d.batch_independent != 1) return NK_ERR_INVALID_ARG;
    if (d.stride_c < 0) return NK_ERR_INVALID_ARG;
    const int64_t str_c = d.stride_c > 0 ? d.stride_c : d.M * d.N;
    const bool indep = d.batch_independent == 1 && nbatch > 1;
    if (indep) {
        const int64_t gran_c = is16(d.out_dtype) ? 8 : 4;
        if (str_c % gran_c) return NK_ERR_MISALIGNED;
        if (str_c < d.M * d.N) return NK_ERR_INVALID_ARG;
        if (nbatch * d.M * d.N >= (1ll << 31)) return NK_ERR_UNSUPPORTED;
    }
    const uint32_t force = d.flags & NK_FLAG_KERNEL_MASK;
    if (force > NK_FLAG_KERNEL_UMMA) return NK_ERR_INVALID_ARG;
    if ((d.flags & NK_FLAG_F32_TENSOR) && d.in_dtype == NK_F32 && force != NK_FLAG_KERNEL_NAIVE) {
        if (force == NK_FLAG_KERNEL_SIMT) return NK_ERR_INVALID_ARG;
        if (nbatch > 1 || d.layout_c != NK_ROW_MAJOR) return NK_ERR_UNSUPPORTED;
        if (d.N % 8 || d.K % 8) return NK_ERR_MISALIGNED;   // the BF16 planes are read by TMA
    }
    if (force != NK_FLAG_KERNEL_NAIVE) {
        if (is16(d.in_dtype) && (d.N % 8 || d.K % 8)) return NK_ERR_MISALIGNED;
        if (d.in_dtype == NK_F32 && (d.N % 4 || d.K % 4)) return NK_ERR_MISALIGNED;
        if (force == NK_FLAG_KERNEL_SIMT && d.in_dtype != NK_F32) return NK_ERR_UNSUPPORTED;
        if (force == NK_FLAG_KERNEL_UMMA && !is16(d.in_dtype) && !is_8bit(d)) return NK_ERR_UNSUPPORTED;
    }

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev <= 0) {
        cudaGetLastError();
        return NK_ERR_DEVICE;
    }
    if (d.device < 0 || d.device >= ndev) return NK_ERR_DEVICE;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, d.device) != cudaSuccess) return NK_ERR_DEVICE;
    if (prop.major != 10) return NK_ERR_DEVICE;

    nk_gemm_s* p = new (std::nothrow) nk_gemm_s();
    if (!p) return NK_ERR_INVALID_ARG;
    memset(p, 0, sizeof(*p));
    p->d = d;
    p->sm_count = prop.multiProcessorCount;
    p->batch = indep ? 1 : static_cast<int>(nbatch);
    p->gemms = indep ? static_cast<int>(nbatch) : 1;
    p->stride_a = str_a;
    p->stride_b = str_b;
    p->stride_c = str_c;
    // a batched matmul whose C's are not contiguous cannot use the flat split-K reduction
    if (indep && str_c != d.M * d.N && ((d.flags >> NK_FLAG_SPLITK_SHIFT) & 0xFF) == 0)
        p->d.flags |= 1u << NK_FLAG_SPLITK_SHIFT;

    DeviceGuard guard(d.device);
    if (guard.err != cudaSuccess) { delete p; return NK_ERR_DEVICE; }
    void* sym = nullptr;
    if (cudaGetSymbolAddress(&sym, g_status_word) != cudaSuccess) { delete p; return NK_ERR_CUDA; }
    p->status_dev = static_cast<unsigned int*>(sym) + (g_next_status_slot.fetch_add(1) % NK_STATUS_SLOTS);
    {
        // the slot may carry the word of a plan that was destroyed without a check
        const unsigned int z = 0;
        if (cudaMemcpy(p->status_dev, &z, sizeof(z), cudaMemcpyHostToDevice) != cudaSuccess) { delete p; return NK_ERR_CUDA; }
    }

    if (d.in_dtype == NK_F32 && (d.flags & NK_FLAG_F32_TENSOR) && force != NK_FLAG_KERNEL_NAIVE) {
        // x = hi + mid + lo in BF16 (to 2^-27 of x); A.B = sum of the nine cross terms, of which the six
        // whose weight is above 2^-25 of |a||b| are kept, smallest first, so the FP32 accumulator of the
        // tensor core sees them in increasing size:  (lo,hi) (hi,lo) (mid,mid) (mid,hi) (hi,mid) (hi,hi)
        p->variant = V_SPLIT3;
        nk_gemm_desc_t id = d;
        id.in_dtype = NK_BF16;
        id.out_dtype = NK_F32;
        id.batch = 6;
        id.batch_independent = 0;
        id.stride_a = static_cast<int64_t>(align_up(static_cast<size_t>(d.M) * d.K, 8));
        id.stride_b = static_cast<int64_t>(align_up(static_cast<size_t>(d.K) * d.N, 8));
        id.flags = d.flags & ~(NK_FLAG_F32_TENSOR | NK_FLAG_KERNEL_MASK | NK_FLAG_SCALAR_FMA);
        nk_gemm_t inner = nullptr;
        const nk_status_t is = nk_gemm_create(&id, &inner);
        if (is != NK_OK) { delete p; return is; }
        inner->status_dev = p->status_dev;   // the plan that the caller holds reports for its inner plan
        inner->bias_f32 = true;
        inner->item_remap = true;
        inner->item_map_a = 0x001102u;   // items 0..5: planes 2 0 1 1 0 0 (0 = hi)
        inner->item_map_b = 0x010120u;   //             planes 0 2 1 0 1 0
        p->inner = inner;
        p->plane_a = id.stride_a;
        p->plane_b = id.stride_b;
        p->ws_repack_bytes = align_up(static_cast<size_t>(p->plane_a) * 6, 256) + align_up(static_cast<size_t>(p->plane_b) * 6, 256);
        p->ws_partial_bytes = nk_gemm_workspace_bytes(inner);
        p->launches = 1 + inner->launches;
        snprintf(p->name, sizeof(p->name), "f32_as_bf16x3_%.100s", inner->name);
        *out = p;
        return NK_OK;
    }
    if (force == NK_FLAG_KERNEL_NAIVE) {
        p->variant = V_NAIVE;
        p->launches = 1;
        snprintf(p->name, sizeof(p->name), "naive");
    } else if (d.in_dtype == NK_F32 && d.M <= 32 && force != NK_FLAG_KERNEL_SIMT && nbatch == 1 && d.beta == 0) {
        p->variant = V_SKINNY;
        choose_skinny(p);
        p->ws_partial_bytes = p->splits > 1 ? static_cast<size_t>(p->splits) * p->gemms * d.M * d.N * 4 : 0;
        p->launches = p->splits > 1 ? 2 : 1;
        snprintf(p->name, sizeof(p->name), "simt_f32_skinny_%dx512_kc%d_splitk%d", d.M <= 16 ? 16 : 32,
                 p->skinny_kc, p->splits);
    } else if (d.in_dtype == NK_F32 && force == NK_FLAG_KERNEL_AUTO && nbatch == 1 && d.K <= SMALL_KMAX &&
               !(d.flags & (0xFu << NK_FLAG_TILE_N_SHIFT)) && !(d.flags & (0xFFu << NK_FLAG_SPLITK_SHIFT)) &&
               static_cast<int64_t>(ceil_div(d.M, SMALL_BM)) * ceil_div(d.N, SMALL_BN) <= 2 * p->sm_count &&
               ceil_div(d.M, SMALL_BM) <= 65535) {
        // a small problem: whole K in shared memory, one launch (see simt_f32_small_kernel)
        p->variant = V_SMALL;
        if (allow_smem(simt_f32_small_kernel, simt_small_smem_bytes(SMALL_KMAX)) != cudaSuccess) { cudaGetLastError(); delete p; return NK_ERR_CUDA; }
        p->splits = 1;
        p->launches = 1;
        snprintf(p->name, sizeof(p->name), "simt_f32_small_32x32_k%d", static_cast<int>(d.K));
    } else if (d.in_dtype == NK_F32) {
        p->variant = V_SIMT;
        if (prepare_simt_attrs() != cudaSuccess) { cudaGetLastError(); delete p; return NK_ERR_CUDA; }
        choose_simt(p);
        p->ws_partial_bytes = p->splits > 1 ? static_cast<size_t>(p->splits) * p->gemms * d.M * d.N * 4 : 0;
        p->launches = p->splits > 1 ? 2 : 1;
        snprintf(p->name, sizeof(p->name), "simt_f32%s_%dx%dx16_splitk%d",
                 (p->simt_tile == 128 && !(d.flags & NK_FLAG_SCALAR_FMA)) ? "x2" : "", p->simt_tile, p->simt_tile,
                 p->splits);
    } else if (is16(d.in_dtype) && d.M <= 64 && force == NK_FLAG_KERNEL_AUTO && nbatch == 1 && d.layout_a == NK_ROW_MAJOR &&
               (d.layout_b == NK_ROW_MAJOR || d.layout_b == NK_TRANSPOSED) && d.layout_c == NK_ROW_MAJOR &&
               !(d.flags & (NK_FLAG_SINGLE_CTA | NK_FLAG_CTA_PAIR | (0xFu << NK_FLAG_TILE_N_SHIFT)))) {
        // few rows of A: the operands swap roles, B's columns become the rows of the MMA (see umma_swap_kernel)
        p->variant = V_SWAP;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess || !fn) {
            delete p;
            return NK_ERR_CUDA;
        }
        p->encode = reinterpret_cast<EncodeTiledFn>(fn);
        p->swap_mp = d.M <= 16 ? 16 : d.M <= 32 ? 32 : 64;
        if (allow_smem(umma_swap_kernel<16, false>, swap_smem_bytes(16, swap_stages(16))) != cudaSuccess ||
            allow_smem(umma_swap_kernel<16, true>, swap_smem_bytes(16, swap_stages(16))) != cudaSuccess ||
            allow_smem(umma_swap_kernel<32, false>, swap_smem_bytes(32, swap_stages(32))) != cudaSuccess ||
            allow_smem(umma_swap_kernel<32, true>, swap_smem_bytes(32, swap_stages(32))) != cudaSuccess ||
            allow_smem(umma_swap_kernel<64, false>, swap_smem_bytes(64, swap_stages(64))) != cudaSuccess ||
            allow_smem(umma_swap_kernel<64, true>, swap_smem_bytes(64, swap_stages(64))) != cudaSuccess) {
            cudaGetLastError();
            delete p;
            return NK_ERR_CUDA;
        }
        p->b_kmajor = d.layout_b == NK_TRANSPOSED;
        // K splits: enough CTAs to pull B from every SM; they meet in one CTA of a cluster (at most 8
        // CTAs; 4 with 64 rows, whose accumulators must fit the stage ring of the receiving CTA)
        const int tiles_n = ceil_div(d.N, 128);
        const int kb_total = ceil_div(d.K, UMMA_BK);
        const int forced_s = (d.flags >> NK_FLAG_SPLITK_SHIFT) & 0xFF;
        const int max_s = p->swap_mp == 64 ? 4 : 8;
        int splits = forced_s > 0 ? forced_s : p->sm_count / tiles_n;
        if (splits > max_s && !(forced_s > 0 && (d.flags & NK_FLAG_SEPARATE_REDUCE))) splits = max_s;
        if (splits > kb_total) splits = kb_total;
        if (splits < 1) splits = 1;
        const int per = ceil_div(kb_total, splits);
        p->splits = ceil_div(kb_total, per);
        p->cluster_reduce = p->splits > 1 && p->splits <= max_s && !(d.flags & NK_FLAG_SEPARATE_REDUCE);
        p->ws_partial_bytes = (p->splits > 1 && !p->cluster_reduce) ? static_cast<size_t>(p->splits) * d.M * d.N * 4 : 0;
        p->launches = (p->splits > 1 && !p->cluster_reduce) ? 2 : 1;
        snprintf(p->name, sizeof(p->name), "umma_swap_128x%dx64_s%d_splitk%d%s%s", p->swap_mp, swap_stages(p->swap_mp), p->splits,
                 p->cluster_reduce ? "_cluster" : "", p->b_kmajor ? "_bt" : "");
    } else {
        p->variant = V_UMMA;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess || !fn) {
            delete p;
            return NK_ERR_CUDA;
        }
        p->encode = reinterpret_cast<EncodeTiledFn>(fn);
        if (prepare_umma_attrs(d.device) != cudaSuccess) { cudaGetLastError(); delete p; return NK_ERR_CUDA; }
        choose_umma(p);
        if (d.layout_b == NK_BLOCKED32) {
            p->b_repack = (d.flags & NK_FLAG_REPACK_B) != 0;
            p->b_vnni_inkernel = !p->b_repack;
        }
        p->b_kmajor = d.layout_b == NK_TRANSPOSED;
        if (p->pair) {
            const bool v = p->b_vnni_inkernel;
            int n = 0;
            cudaError_t oe = p->bn == 256
                ? (v ? pair_occupancy<256, 6, true>(&n) : pair_occupancy<256, 6, false>(&n))
                : (v ? pair_occupancy<128, 8, true>(&n) : pair_occupancy<128, 8, false>(&n));
            if (oe != cudaSuccess || n <= 0) { cudaGetLastError(); delete p; return NK_ERR_CUDA; }
            p->max_pairs = n;
        }
        if (p->cluster_reduce) {
            // every cluster of the plan must be resident at once (one unit per CTA): ask the driver
            int n = 0;
            const int clusters = p->gemms * ceil_div(d.M, p->pair ? 2 * UMMA_BM : UMMA_BM) * ceil_div(d.N, p->bn);
            if (launch_cluster(p, UmmaParams(), 0, p->splits, nullptr, &n) != cudaSuccess || n < clusters) {
                cudaGetLastError();
                p->cluster_reduce = false;
            }
        }
        // Ragged last wave (stream-K): when the tiles left after the last full wave do not fill the
        // pairs, their k-blocks are shared out evenly over all the pairs, so that the wave takes a
        // fraction of a K loop; worth it when the K loop saved outweighs the small reduce kernel and
        // the partials (FP32, written and read once).  NK_FLAG_TAIL_SPLIT forces equal cuts instead.
        p->tail_from = -1;
        p->tail_splits = 0;
        p->sk_share = p->sk_max_segs = 0;
        if (p->pair && p->splits == 1 && p->gemms == 1 && !(d.flags & NK_FLAG_NO_TAIL_SPLIT)) {
            const int tiles = ceil_div(d.M, 2 * UMMA_BM) * ceil_div(d.N, p->bn);
            const int kb_total = p->batch * ceil_div(d.K, kblock(d));
            const int P = p->max_pairs;
            const int tail = tiles % P;
            int forced_tail = (d.flags >> NK_FLAG_TAIL_SPLIT_SHIFT) & 0xF;
            bool forced_even = forced_tail == 15;            // the even share, whatever the cost model says
            if (forced_tail >= 2 && forced_tail <= 8 && tail * forced_tail > P) forced_even = true;   // equal cuts would need more pairs than there are
            if (forced_tail < 2 || forced_tail > 8 || forced_tail > kb_total || tail * forced_tail > P) forced_tail = 0;
            if (tiles > P && tail > 0 && kb_total >= 2) {
                int share = forced_tail ? ceil_div(kb_total, forced_tail) : ceil_div(static_cast<int64_t>(tail) * kb_total, P);
                if (!forced_tail && !forced_even && share < 4) share = kb_total < 4 ? kb_total : 4;   // shorter ranges are all overhead
                const int segments = tail + ceil_div(static_cast<int64_t>(tail) * kb_total, share);   // at most: every pair, every tile boundary
                const double t_kb = p->bn == 256 ? 0.385 : 0.35;
                const double slab_bytes = static_cast<double>(segments) * 2 * UMMA_BM * p->bn * 4;
                const double saved_us = (kb_total - share) * t_kb;
                // measured: ~10 us for 18 MB of partials (they stay in L2); a pair whose range straddles two tiles
                // drains two accumulators
                const double cost_us = 5.5 + 2.0 * slab_bytes / 7.0e6 + p->bn / 32 * 0.5;
                if (share < kb_total && (saved_us > cost_us || forced_tail || forced_even)) {
                    p->tail_from = tiles - tail;
                    p->tail_splits = forced_tail;
                    p->sk_share = share;
                    p->sk_max_segs = (kb_total + share - 2) / share + 1;
                }
            }
        }
        p->tma_store = d.layout_c == NK_ROW_MAJOR && d.beta == 0 && (p->splits == 1 || p->cluster_reduce) &&
                       !(d.flags & NK_FLAG_LSU_STORE);
        p->ws_repack_bytes = p->b_repack ? align_up(static_cast<size_t>(d.K) * d.N * 2, 256) : 0;
        p->ws_partial_bytes = (p->splits > 1 && !p->cluster_reduce) ? static_cast<size_t>(p->splits) * p->gemms * d.M * d.N * 4 : 0;
        if (p->tail_from >= 0) {
            const int tiles = ceil_div(d.M, 2 * UMMA_BM) * ceil_div(d.N, p->bn);
            p->ws_partial_bytes = static_cast<size_t>(tiles - p->tail_from) * p->sk_max_segs * 2 * UMMA_BM * p->bn * 4;
        }
        p->launches = 1 + ((p->splits > 1 && !p->cluster_reduce) || p->tail_from >= 0 ? 1 : 0) + (p->b_repack ? 1 : 0);
        snprintf(p->name, sizeof(p->name), "umma_bf16_%s%dx%d_s%d_splitk%d%s%s%s",
                 p->pair ? "pair_256x" : "128x", p->bn, kblock(d), p->stages,
                 p->splits, p->cluster_reduce ? "_cluster" : "", d.layout_a == NK_BLOCKED32 ? "_ablk" : "",
                 p->b_vnni_inkernel ? "_bvnni" : p->b_repack ? "_brepack" : p->b_kmajor ? "_bt" : "");
    }
    if (p->batch > 1 || p->gemms > 1 || d.beta) {
        const size_t len = strlen(p->name);
        if (p->gemms > 1) snprintf(p->name + len, sizeof(p->name) - len, "_bmm%d%s", p->gemms, d.beta ? "_beta1" : "");
        else snprintf(p->name + len, sizeof(p->name) - len, "_br%d%s", p->batch, d.beta ? "_beta1" : "");
    }
    if (d.layout_c == NK_BLOCKED32) {
        const size_t len = strlen(p->name);
        snprintf(p->name + len, sizeof(p->name) - len, "_cblk");
    }
    if (p->variant == V_UMMA && p->tail_from >= 0) {
        const size_t len = strlen(p->name);
        if (p->tail_splits) snprintf(p->name + len, sizeof(p->name) - len, "_tail%d", p->tail_splits);
        else snprintf(p->name + len, sizeof(p->name) - len, "_streamk%d", p->sk_share);
    }
    if (d.in_dtype == NK_F16) {
        const size_t len = strlen(p->name);
        snprintf(p->name + len, sizeof(p->name) - len, "_f16");
    }
    if (is_f8(d)) {
        const size_t len = strlen(p->name);
        snprintf(p->name + len, sizeof(p->name) - len, d.in_dtype == NK_E4M3 ? "_e4m3" : "_e5m2");
    }
    if (d.in_dtype == NK_S8) {
        const size_t len = strlen(p->name);
        snprintf(p->name + len, sizeof(p->name) - len, d.out_dtype == NK_F32 ? "_s8_dequant" : "_s8");
    }
    // split-K partials are laid out [split][gemm][M][N] and reduced as one flat array: that
    // needs the C of a batched matmul to be contiguous
    if (p->gemms > 1 && p->splits > 1 && p->stride_c != d.M * d.N && !p->cluster_reduce) {
        delete p;
        *out = nullptr;
        return NK_ERR_UNSUPPORTED;
    }
    *out = p;
    return NK_OK;
}

size_t nk_gemm_workspace_bytes(nk_gemm_t p) { return p ? p->ws_repack_bytes + p->ws_partial_bytes : 0; }

int nk_gemm_launches_per_run(nk_gemm_t p) { return p ? p->launches : 0; }

const char* nk_gemm_kernel_name(nk_gemm_t p) { return p ? p->name : ""; }

const char* nk_gemm_last_cuda_error(nk_gemm_t p) { return p ? p->cuda_err : ""; }

nk_status_t nk_gemm_run(nk_gemm_t p, const void* A, const void* B, const void* bias, void* C,
                        void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!p || !A || !B || !C) return NK_ERR_INVALID_ARG;
    const nk_gemm_desc_t& d = p->d;
    if (d.epilogue != NK_EPI_NONE && !bias) return NK_ERR_INVALID_ARG;
    auto mis = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) != 0; };
    if (mis(A) || mis(B) || mis(C) || (bias && mis(bias)) || (workspace && mis(workspace)))
        return NK_ERR_MISALIGNED;
    const size_t need = p->ws_repack_bytes + p->ws_partial_bytes;
    if (need > 0 && (!workspace || workspace_bytes < need)) return NK_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard(d.device);
    if (guard.err != cudaSuccess) { set_err(p, "cudaSetDevice", guard.err); return NK_ERR_DEVICE; }
    cudaError_t e = cudaSuccess;

    if (p->variant == V_NAIVE) {
        NaiveParams np = {static_cast<int>(d.M), static_cast<int>(d.N), static_cast<int>(d.K),
                          is16(d.in_dtype), is16(d.out_dtype), d.layout_a == NK_BLOCKED32,
                          d.layout_b == NK_BLOCKED32, d.epilogue, p->batch, d.beta, p->stride_a, p->stride_b,
                          p->gemms, p->stride_c, d.layout_c == NK_BLOCKED32, A, B, bias, C, d.in_dtype == NK_F16};
        dim3 grid(ceil_div(d.N, 128), static_cast<unsigned>(d.M), static_cast<unsigned>(p->gemms));
        if (d.M > 65535) return NK_ERR_UNSUPPORTED;
        naive_gemm_kernel<<<grid, 128, 0, st>>>(np);
        e = cudaGetLastError();
        if (e != cudaSuccess) { set_err(p, "naive launch", e); return NK_ERR_CUDA; }
        return NK_OK;
    }

    if (p->variant == V_SPLIT3) {
        uint8_t* w8 = static_cast<uint8_t*>(workspace);
        uint16_t* pa = reinterpret_cast<uint16_t*>(w8);
        uint16_t* pb = reinterpret_cast<uint16_t*>(w8 + align_up(static_cast<size_t>(p->plane_a) * 6, 256));
        const long long na = static_cast<long long>(d.M) * d.K, nb = static_cast<long long>(d.K) * d.N;
        auto blocks = [&](long long n) {
            const long long want = (n / 4 + 255) / 256;
            const long long cap = static_cast<long long>(p->sm_count) * 16;
            return static_cast<unsigned>(want < cap ? (want > 0 ? want : 1) : cap);
        };
        const SplitOperand sa = {static_cast<const float*>(A), pa, na, p->plane_a};
        const SplitOperand sb = {static_cast<const float*>(B), pb, nb, p->plane_b};
        split_f32_bf16x3_kernel<<<blocks(na) + blocks(nb), 256, 0, st>>>(sa, sb, blocks(na));
        e = cudaGetLastError();
        if (e != cudaSuccess) { set_err(p, "split launch", e); return NK_ERR_CUDA; }
        const nk_status_t rs = nk_gemm_run(p->inner, pa, pb, bias, C, p->ws_partial_bytes ? w8 + p->ws_repack_bytes : nullptr,
                                           p->ws_partial_bytes, cuda_stream);
        if (rs != NK_OK) memcpy(p->cuda_err, p->inner->cuda_err, sizeof(p->cuda_err));
        return rs;
    }

    uint8_t* ws = static_cast<uint8_t*>(workspace);
    float* partial = p->ws_partial_bytes ? reinterpret_cast<float*>(ws + p->ws_repack_bytes) : nullptr;

    if (p->variant == V_SMALL) {
        SmallParams mp = {static_cast<int>(d.M), static_cast<int>(d.N), static_cast<int>(d.K), d.beta, d.epilogue,
                          static_cast<const float*>(A), static_cast<const float*>(B), static_cast<const float*>(bias),
                          static_cast<float*>(C)};
        dim3 grid(ceil_div(d.N, SMALL_BN), ceil_div(d.M, SMALL_BM));
        simt_f32_small_kernel<<<grid, SMALL_THREADS, simt_small_smem_bytes(static_cast<int>(d.K)), st>>>(mp);
        e = cudaGetLastError();
        if (e != cudaSuccess) { set_err(p, "small launch", e); return NK_ERR_CUDA; }
    } else if (p->variant == V_SKINNY) {
        SkinnyParams kp = {static_cast<int>(d.M), static_cast<int>(d.N), static_cast<int>(d.K), p->skinny_kc,
                           p->splits, d.epilogue, static_cast<const float*>(A), static_cast<const float*>(B),
                           static_cast<const float*>(bias), static_cast<float*>(C), partial};
        dim3 grid(ceil_div(d.N, SKINNY_COLS), p->splits);
        if (d.M <= 16) simt_f32_skinny_kernel<16><<<grid, SKINNY_THREADS, 0, st>>>(kp);
        else simt_f32_skinny_kernel<32><<<grid, SKINNY_THREADS, 0, st>>>(kp);
        e = cudaGetLastError();
        if (e != cudaSuccess) { set_err(p, "skinny launch", e); return NK_ERR_CUDA; }
    } else if (p->variant == V_SIMT) {
        SimtParams sp = {static_cast<int>(d.M), static_cast<int>(d.N), static_cast<int>(d.K), p->splits,
                         p->kt_per_split, p->batch, ceil_div(d.K, SIMT_BK), p->stride_a, p->stride_b, d.beta,
                         p->gemms, p->stride_c, d.epilogue, static_cast<const float*>(A),
                         static_cast<const float*>(B), static_cast<const float*>(bias),
                         static_cast<float*>(C), partial};
        e = launch_simt(p, sp, st);
        if (e != cudaSuccess) { set_err(p, "simt launch", e); return NK_ERR_CUDA; }
    } else if (p->variant == V_SWAP) {
        nk_status_t s = encode_maps(p, A, B);
        if (s != NK_OK) return s;
        SwapParams sp;
        memset(&sp, 0, sizeof(sp));
        sp.M = static_cast<int>(d.M); sp.N = static_cast<int>(d.N); sp.K = static_cast<int>(d.K);
        sp.tiles_n = ceil_div(d.N, 128);
        sp.splits = p->splits;
        sp.kb_total = ceil_div(d.K, UMMA_BK);
        sp.kb_per_split = ceil_div(sp.kb_total, p->splits);
        sp.cluster = p->cluster_reduce ? 1 : 0;
        sp.b_3d = p->b_3d ? 1 : 0;
        sp.b_kmajor = p->b_kmajor ? 1 : 0;
        sp.epilogue = d.epilogue;
        sp.out_bf16 = is16(d.out_dtype);
        sp.f16 = d.in_dtype == NK_F16;
        sp.bias_f32 = 0;
        sp.beta = d.beta;
        sp.idesc = make_idesc_swap(p->swap_mp, !p->b_kmajor, d.in_dtype == NK_F16);
        sp.bias = bias;
        sp.C = C;
        sp.partial = partial;
        sp.status = p->status_dev;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(sp.tiles_n * p->splits));
        cfg.blockDim = dim3(192);
        cfg.dynamicSmemBytes = static_cast<size_t>(swap_smem_bytes(p->swap_mp, swap_stages(p->swap_mp)));
        cfg.stream = st;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = static_cast<unsigned>(p->cluster_reduce ? p->splits : 1);
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        const bool cl = p->cluster_reduce;
        if (p->swap_mp == 16) e = cl ? cudaLaunchKernelEx(&cfg, umma_swap_kernel<16, true>, p->tmap_a, p->tmap_b, sp)
                                     : cudaLaunchKernelEx(&cfg, umma_swap_kernel<16, false>, p->tmap_a, p->tmap_b, sp);
        else if (p->swap_mp == 32) e = cl ? cudaLaunchKernelEx(&cfg, umma_swap_kernel<32, true>, p->tmap_a, p->tmap_b, sp)
                                          : cudaLaunchKernelEx(&cfg, umma_swap_kernel<32, false>, p->tmap_a, p->tmap_b, sp);
        else e = cl ? cudaLaunchKernelEx(&cfg, umma_swap_kernel<64, true>, p->tmap_a, p->tmap_b, sp)
                    : cudaLaunchKernelEx(&cfg, umma_swap_kernel<64, false>, p->tmap_a, p->tmap_b, sp);
        if (e != cudaSuccess) { set_err(p, "swap launch", e); return NK_ERR_CUDA; }
    } else {
        const void* Buse = B;
        if (p->b_repack) {
            dim3 grid(static_cast<unsigned>(d.K / 32), static_cast<unsigned>(d.N / 32));
            unpack_vnni_b_kernel<<<grid, 256, 0, st>>>(static_cast<const uint32_t*>(B),
                                                       reinterpret_cast<uint16_t*>(ws),
                                                       static_cast<int>(d.N), static_cast<int>(d.K));
            e = cudaGetLastError();
            if (e != cudaSuccess) { set_err(p, "unpack launch", e); return NK_ERR_CUDA; }
            Buse = ws;
        }
        nk_status_t s = encode_maps(p, A, Buse);
        if (s != NK_OK) return s;
        if ((s = encode_c_map(p, C)) != NK_OK) return s;
        UmmaParams up;
        memset(&up, 0, sizeof(up));
        up.M = static_cast<int>(d.M); up.N = static_cast<int>(d.N); up.K = static_cast<int>(d.K);
        up.tiles_m = ceil_div(d.M, p->pair ? 2 * UMMA_BM : UMMA_BM);
        up.tiles_n = ceil_div(d.N, p->bn);
        up.splits = p->splits;
        up.kb_per_item = ceil_div(d.K, kblock(d));
        up.kb_total = p->batch * up.kb_per_item;
        up.beta = d.beta;
        up.gemms = p->gemms;
        up.stride_c = p->stride_c;
        up.c_blocked = d.layout_c == NK_BLOCKED32;
        up.tma_store = p->tma_store ? 1 : 0;
        up.cluster_reduce = p->cluster_reduce ? 1 : 0;
        up.kb_per_split = ceil_div(up.kb_total, p->splits);
        up.group_m = p->group_m;
        up.serpentine = p->serpentine ? 1 : 0;
        up.k_serpentine = (p->k_serpentine && p->pair && p->splits == 1 && p->batch == 1) ? 1 : 0;
        up.a_blocked = d.layout_a == NK_BLOCKED32;
        up.b_3d = p->b_3d ? 1 : 0;
        up.b_kmajor = p->b_kmajor ? 1 : 0;
        up.epilogue = d.epilogue;
        up.out_bf16 = is16(d.out_dtype);
        up.idesc = make_idesc(p->pair ? 2 * UMMA_BM : UMMA_BM, p->bn, !p->b_vnni_inkernel && !p->b_kmajor, d.in_dtype == NK_F16, is_s8(d),
                              d.in_dtype == NK_E4M3 ? 0 : d.in_dtype == NK_E5M2 ? 1 : -1);
        up.f16 = d.in_dtype == NK_F16;
        up.bias = bias;
        up.C = C;
        up.partial = partial;
        up.status = p->status_dev;
        up.bias_f32 = (p->bias_f32 || is_8bit(d)) ? 1 : 0;
        up.dequant = (is_s8(d) && d.out_dtype == NK_F32) ? 1 : 0;
        up.scale = d.scale;
        up.acc_s32 = is_s8(d) ? 1 : 0;
        up.item_remap = p->item_remap ? 1 : 0;
        up.item_map_a = p->item_map_a;
        up.item_map_b = p->item_map_b;
        up.tail_from = p->tail_from;
        up.sk_share = p->sk_share;
        up.sk_max_segs = p->sk_max_segs;
        // (tail mode: more tiles than pairs, so every pair is launched; each adds up to two tail segments to its whole tiles)
        const int units = p->tail_from >= 0 ? p->tail_from + 2 * p->max_pairs : up.gemms * up.tiles_m * up.tiles_n * up.splits;
        if (p->cluster_reduce) {
            e = launch_cluster(p, up, units, p->splits, st, nullptr);
        } else if (p->pair) {
            const int pairs = units < p->max_pairs ? units : p->max_pairs;
            e = launch_pair(p, up, pairs, st);
        } else {
            const int grid = units < p->sm_count ? units : p->sm_count;
            e = launch_umma(p, up, grid, st);
        }
        if (e != cudaSuccess) { set_err(p, "umma launch", e); return NK_ERR_CUDA; }
    }

    if (p->variant == V_UMMA && p->tail_from >= 0) {
        const int tiles_m = ceil_div(d.M, 2 * UMMA_BM), tiles_n = ceil_div(d.N, p->bn);
        TailReduceParams tp = {static_cast<int>(d.M), static_cast<int>(d.N), 2 * UMMA_BM, p->bn, tiles_m, tiles_n, p->group_m,
                               p->tail_from, p->serpentine ? 1 : 0, p->batch * ceil_div(d.K, kblock(d)), p->sk_share, p->sk_max_segs,
                               d.epilogue, (p->bias_f32 || is_8bit(d)) ? 0 : 1, is16(d.out_dtype), d.beta,
                               d.layout_c == NK_BLOCKED32, d.in_dtype == NK_F16, partial, bias, C,
                               is_s8(d) ? 1 : 0, (is_s8(d) && d.out_dtype == NK_F32) ? 1 : 0, d.scale};
        const int quads = 2 * UMMA_BM * p->bn / 4;
        dim3 grid(static_cast<unsigned>((quads + 255) / 256), static_cast<unsigned>(tiles_m * tiles_n - p->tail_from));
        tail_reduce_kernel<<<grid, 256, 0, st>>>(tp);
        e = cudaGetLastError();
        if (e != cudaSuccess) { set_err(p, "tail reduce launch", e); return NK_ERR_CUDA; }
    }
    if (p->splits > 1 && !p->cluster_reduce) {
        ReduceParams rp = {static_cast<size_t>(p->gemms) * d.M * d.N, static_cast<int>(d.N), p->splits, d.epilogue,
                           is16(d.in_dtype) && !p->bias_f32, is16(d.out_dtype), d.beta, d.layout_c == NK_BLOCKED32,
                           static_cast<int>(d.M), partial, bias, C, d.in_dtype == NK_F16,
                           is_s8(d) ? 1 : 0, (is_s8(d) && d.out_dtype == NK_F32) ? 1 : 0, d.scale};
        const size_t quads = rp.MN / 4;
        splitk_reduce_kernel<<<static_cast<unsigned>((quads + 255) / 256), 256, 0, st>>>(rp);
        e = cudaGetLastError();
        if (e != cudaSuccess) { set_err(p, "reduce launch", e); return NK_ERR_CUDA; }
    }
    return NK_OK;
}

nk_status_t nk_gemm_run_host(nk_gemm_t p, const void* hA, const void* hB, const void* hbias, void* hC,
                             void* dA, void* dB, void* dbias, void* dC, void* workspace,
                             size_t workspace_bytes, void* cuda_stream) {
    if (!p || !hA || !hB || !hC || !dA || !dB || !dC) return NK_ERR_INVALID_ARG;
    const nk_gemm_desc_t& d = p->d;
    if (d.epilogue != NK_EPI_NONE && (!hbias || !dbias)) return NK_ERR_INVALID_ARG;
    const size_t ein = is_8bit(d) ? 1 : is16(d.in_dtype) ? 2 : 4, eout = is16(d.out_dtype) ? 2 : 4;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    DeviceGuard guard(d.device);
    if (guard.err != cudaSuccess) { set_err(p, "cudaSetDevice", guard.err); return NK_ERR_DEVICE; }
    cudaError_t e;
    // Large single GEMMs: the host link, not the GPU, bounds this call.  A travels in eight chunks of
    // rows, B in four panels of columns (one when N does not divide), C comes back as the 8 x 4
    // blocks they span: uploads alternate between the two operands, every block is multiplied on
    // the caller's stream as soon as its row chunk and its column panel have arrived, and goes
    // down on a second copy stream while later uploads are still running (PCIe is full duplex).
    // On the device the panels of B and the blocks of C are dense (the staging buffers are
    // scratch); the copies convert between that and the row-major host matrices.
    constexpr int kRowChunks = 8, kMaxPanels = 4;
    if (d.beta == 0 && p->batch == 1 && p->gemms == 1 && d.layout_c == NK_ROW_MAJOR && d.M % (kRowChunks * 256) == 0 &&
        2.0 * d.M * d.N * d.K >= 2.0e10 && !(d.flags & NK_FLAG_KERNEL_MASK)) {
        if (!p->chunk_plan && !p->chunk_tried) {
            p->chunk_tried = true;
            const int panels = d.N % (kMaxPanels * 256) == 0 ? kMaxPanels : 1;
            nk_gemm_desc_t cd = d;
            cd.M = d.M / kRowChunks;
            cd.N = d.N / panels;
            cd.flags = (d.flags & ~(0xFFu << NK_FLAG_SPLITK_SHIFT)) | (1u << NK_FLAG_SPLITK_SHIFT) | NK_FLAG_NO_TAIL_SPLIT;
            nk_gemm_t cp = nullptr;
            nk_status_t cs = nk_gemm_create(&cd, &cp);
            if (cs == NK_OK) cp->status_dev = p->status_dev;   // the caller's plan reports for its chunk plan
            if (cs == NK_OK && nk_gemm_workspace_bytes(cp) == 0) {
                bool ok = cudaStreamCreateWithFlags(&p->h2d_stream, cudaStreamNonBlocking) == cudaSuccess &&
                          cudaStreamCreateWithFlags(&p->d2h_stream, cudaStreamNonBlocking) == cudaSuccess &&
                          cudaEventCreateWithFlags(&p->ev_start, cudaEventDisableTiming) == cudaSuccess &&
                          cudaEventCreateWithFlags(&p->ev_done, cudaEventDisableTiming) == cudaSuccess;
                for (int i = 0; ok && i < kRowChunks + kMaxPanels; ++i)
                    ok = cudaEventCreateWithFlags(&p->ev_up[i], cudaEventDisableTiming) == cudaSuccess;
                for (int i = 0; ok && i < kRowChunks * kMaxPanels; ++i)
                    ok = cudaEventCreateWithFlags(&p->ev_g[i], cudaEventDisableTiming) == cudaSuccess;
                if (ok) {
                    p->chunk_plan = cp;
                    p->chunk_rows = static_cast<int>(cd.M);
                    p->chunk_panels = panels;
                } else {
                    cudaGetLastError();
                    nk_gemm_destroy(cp);
                }
            } else if (cp) {
                nk_gemm_destroy(cp);
            }
        }
        if (p->chunk_plan) {
            const size_t ein_b = is_8bit(d) ? 1 : is16(d.in_dtype) ? 2 : 4, eout_b = is16(d.out_dtype) ? 2 : 4;
            const int panels = p->chunk_panels;
            const size_t rows = static_cast<size_t>(p->chunk_rows), cols = static_cast<size_t>(d.N) / panels;
            const size_t a_chunk = rows * d.K * ein_b;                         // also right for blocked A
            const size_t b_panel = static_cast<size_t>(d.K) * cols * ein_b;     // dense on the device
            const size_t c_block = rows * cols * eout_b;                       // dense on the device
            const bool has_bias = d.epilogue != NK_EPI_NONE;
            const size_t ebias_b = is_8bit(d) ? 4 : ein_b;   // 8-bit operands come with an FP32 bias
            const bool b_rows_strided = d.layout_b == NK_ROW_MAJOR && panels > 1;   // a blocked B panel is contiguous
            bool ok = cudaEventRecord(p->ev_start, st) == cudaSuccess &&
                      cudaStreamWaitEvent(p->h2d_stream, p->ev_start, 0) == cudaSuccess &&
                      cudaStreamWaitEvent(p->d2h_stream, p->ev_start, 0) == cudaSuccess &&
                      (!has_bias || cudaMemcpyAsync(dbias, hbias, static_cast<size_t>(d.N) * ebias_b, cudaMemcpyHostToDevice, p->h2d_stream) == cudaSuccess);
            int na = 0, nb = 0, nup = 0, ng = 0;     // row chunks and panels on the device; uploads and blocks so far
            while (ok && (na < kRowChunks || nb < panels)) {
                // A0, B0, then B and A in turn until one runs out
                const bool up_a = nb >= panels || (na < kRowChunks && na < nb + (na == 0 ? 1 : 0));
                if (up_a) {
                    ok = cudaMemcpyAsync(static_cast<char*>(dA) + na * a_chunk, static_cast<const char*>(hA) + na * a_chunk, a_chunk,
                                         cudaMemcpyHostToDevice, p->h2d_stream) == cudaSuccess;
                } else if (b_rows_strided) {
                    ok = cudaMemcpy2DAsync(static_cast<char*>(dB) + nb * b_panel, cols * ein_b,
                                           static_cast<const char*>(hB) + nb * cols * ein_b, static_cast<size_t>(d.N) * ein_b,
                                           cols * ein_b, static_cast<size_t>(d.K), cudaMemcpyHostToDevice, p->h2d_stream) == cudaSuccess;
                } else {
                    ok = cudaMemcpyAsync(static_cast<char*>(dB) + nb * b_panel, static_cast<const char*>(hB) + nb * b_panel, b_panel,
                                         cudaMemcpyHostToDevice, p->h2d_stream) == cudaSuccess;
                }
                ok = ok && cudaEventRecord(p->ev_up[nup], p->h2d_stream) == cudaSuccess &&
                     cudaStreamWaitEvent(st, p->ev_up[nup], 0) == cudaSuccess;
                ++nup;
                if (!ok) break;
                // the blocks this upload completes: a new row chunk meets every panel present, and vice versa
                const int i0 = up_a ? na : 0, i1 = up_a ? na + 1 : na;
                const int j0 = up_a ? 0 : nb, j1 = up_a ? nb : nb + 1;
                if (up_a) ++na; else ++nb;
                for (int i = i0; ok && i < i1; ++i)
                    for (int j = j0; ok && j < j1; ++j) {
                        char* dC_ij = static_cast<char*>(dC) + (static_cast<size_t>(i) * panels + j) * c_block;
                        nk_status_t rs = nk_gemm_run(p->chunk_plan, static_cast<char*>(dA) + i * a_chunk,
                                                     static_cast<char*>(dB) + j * b_panel,
                                                     has_bias ? static_cast<char*>(dbias) + j * cols * ebias_b : nullptr, dC_ij,
                                                     nullptr, 0, cuda_stream);
                        if (rs != NK_OK) {
                            snprintf(p->cuda_err, sizeof(p->cuda_err), "block %d,%d: %s", i, j, nk_gemm_last_cuda_error(p->chunk_plan));
                            cudaStreamSynchronize(p->h2d_stream);
                            cudaStreamSynchronize(p->d2h_stream);
                            cudaStreamSynchronize(st);
                            return rs;
                        }
                        char* hC_ij = static_cast<char*>(hC) + (static_cast<size_t>(i) * rows * d.N + j * cols) * eout_b;
                        ok = cudaEventRecord(p->ev_g[ng], st) == cudaSuccess &&
                             cudaStreamWaitEvent(p->d2h_stream, p->ev_g[ng], 0) == cudaSuccess &&
                             cudaMemcpy2DAsync(hC_ij, static_cast<size_t>(d.N) * eout_b, dC_ij, cols * eout_b, cols * eout_b, rows,
                                               cudaMemcpyDeviceToHost, p->d2h_stream) == cudaSuccess;
                        ++ng;
                    }
            }
            ok = ok && cudaEventRecord(p->ev_done, p->d2h_stream) == cudaSuccess &&
                 cudaStreamWaitEvent(st, p->ev_done, 0) == cudaSuccess;
            e = cudaStreamSynchronize(st);
            if (!ok || e != cudaSuccess) {
                cudaStreamSynchronize(p->h2d_stream);
                cudaStreamSynchronize(p->d2h_stream);
                set_err(p, "pipelined host run", e != cudaSuccess ? e : cudaGetLastError());
                return NK_ERR_CUDA;
            }
            return NK_OK;
        }
    }
    const size_t items = static_cast<size_t>(p->batch) * p->gemms;
    const size_t a_elems = (items - 1) * p->stride_a + static_cast<size_t>(d.M) * d.K;
    const size_t b_elems = (items - 1) * p->stride_b + static_cast<size_t>(d.K) * d.N;
    const size_t c_elems = static_cast<size_t>(p->gemms - 1) * p->stride_c + static_cast<size_t>(d.M) * d.N;
    if (d.beta && (e = cudaMemcpyAsync(dC, hC, eout * c_elems, cudaMemcpyHostToDevice, st)) != cudaSuccess) {
        set_err(p, "H2D copy", e);
        return NK_ERR_CUDA;
    }
    if ((e = cudaMemcpyAsync(dA, hA, ein * a_elems, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
        (e = cudaMemcpyAsync(dB, hB, ein * b_elems, cudaMemcpyHostToDevice, st)) != cudaSuccess) {
        set_err(p, "H2D copy", e);
        return NK_ERR_CUDA;
    }
    if (d.epilogue != NK_EPI_NONE &&
        (e = cudaMemcpyAsync(dbias, hbias, (is_8bit(d) ? 4 : ein) * d.N, cudaMemcpyHostToDevice, st)) != cudaSuccess) {
        set_err(p, "H2D copy", e);
        return NK_ERR_CUDA;
    }
    nk_status_t s = nk_gemm_run(p, dA, dB, d.epilogue != NK_EPI_NONE ? dbias : nullptr, dC, workspace,
                                workspace_bytes, cuda_stream);
    if (s != NK_OK) return s;
    if ((e = cudaMemcpyAsync(hC, dC, eout * c_elems, cudaMemcpyDeviceToHost, st)) != cudaSuccess ||
        (e = cudaStreamSynchronize(st)) != cudaSuccess) {
        set_err(p, "D2H copy / sync", e);
        return NK_ERR_CUDA;
    }
    return NK_OK;
}

// ---------------------------------------------------------------------------
// Scratch for callers that cannot allocate: a fixed array inside the library
// image.  In host code the symbol below is only a handle, not a device address;
// the address each device gave it is looked up once per device and cached.
static __device__ __align__(256) unsigned char g_static_scratch[NK_STATIC_SCRATCH_BYTES];

namespace nk {
constexpr int kMaxDevices = 64;
static std::mutex g_scratch_mu;
static void* g_scratch_addr[kMaxDevices];   // device address of g_static_scratch, per device
}  // namespace nk

nk_status_t nk_gemm_run_static(nk_gemm_t p, const void* A, const void* B, const void* bias, void* C,
                               void* cuda_stream) {
    if (!p) return NK_ERR_INVALID_ARG;
    const size_t need = p->ws_repack_bytes + p->ws_partial_bytes;
    if (need > NK_STATIC_SCRATCH_BYTES) {
        snprintf(p->cuda_err, sizeof(p->cuda_err),
                 "plan needs %zu bytes of scratch; the built-in array holds %u", need,
                 (unsigned)NK_STATIC_SCRATCH_BYTES);
        return NK_ERR_WORKSPACE;
    }
    if (need == 0) return nk_gemm_run(p, A, B, bias, C, nullptr, 0, cuda_stream);
    const int dev = p->d.device;
    if (dev < 0 || dev >= kMaxDevices) return NK_ERR_DEVICE;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_scratch_mu);
        if (!g_scratch_addr[dev]) {
            DeviceGuard guard(dev);   // the lookup answers for the current device
            if (guard.err != cudaSuccess) { set_err(p, "cudaSetDevice", guard.err); return NK_ERR_DEVICE; }
            void* addr = nullptr;
            cudaError_t e = cudaGetSymbolAddress(&addr, g_static_scratch);
            if (e != cudaSuccess || !addr) { set_err(p, "cudaGetSymbolAddress", e); return NK_ERR_CUDA; }
            g_scratch_addr[dev] = addr;
        }
        scratch = g_scratch_addr[dev];
    }
    return nk_gemm_run(p, A, B, bias, C, scratch, NK_STATIC_SCRATCH_BYTES, cuda_stream);
}

nk_status_t nk_gemm_check(nk_gemm_t p) {
    if (!p) return NK_ERR_INVALID_ARG;
    DeviceGuard guard(p->d.device);
    if (guard.err != cudaSuccess) return NK_ERR_DEVICE;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { set_err(p, "cudaDeviceSynchronize", e); return NK_ERR_CUDA; }
    unsigned int w = 0;
    e = cudaMemcpy(&w, p->status_dev, sizeof(w), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { set_err(p, "status read", e); return NK_ERR_CUDA; }
    if (w != 0) {
        snprintf(p->cuda_err, sizeof(p->cuda_err), "device wait gave up, code 0x%x", w);
        unsigned int z = 0;
        cudaMemcpy(p->status_dev, &z, sizeof(z), cudaMemcpyHostToDevice);
        return NK_ERR_TIMEOUT;
    }
    return NK_OK;
}

nk_status_t nk_gemm_selftest_timeout(nk_gemm_t p, void* cuda_stream) {
    if (!p) return NK_ERR_INVALID_ARG;
    DeviceGuard guard(p->d.device);
    if (guard.err != cudaSuccess) return NK_ERR_DEVICE;
    wait_timeout_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(p->status_dev, 1ll << 22);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_err(p, "probe launch", e); return NK_ERR_CUDA; }
    return NK_OK;
}

nk_status_t nk_quantize_s8(const float* x, int8_t* q, size_t n, float inv_scale, int device, void* cuda_stream) {
    if (!x || !q) return NK_ERR_INVALID_ARG;
    if (n == 0) return NK_OK;
    if (n >= 4 && (reinterpret_cast<uintptr_t>(x) & 15u)) return NK_ERR_MISALIGNED;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) { cudaGetLastError(); return NK_ERR_DEVICE; }
    DeviceGuard guard(device);
    if (guard.err != cudaSuccess) return NK_ERR_DEVICE;
    const size_t blocks = (n / 4 + 1 + 255) / 256;
    if (blocks > 0x7FFFFFFFull) return NK_ERR_UNSUPPORTED;
    quantize_s8_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(x, q, n, inv_scale);
    return cudaGetLastError() == cudaSuccess ? NK_OK : NK_ERR_CUDA;
}

nk_status_t nk_gemm_destroy(nk_gemm_t p) {
    if (p && p->inner) nk_gemm_destroy(p->inner);
    if (p && p->chunk_plan) {
        DeviceGuard guard(p->d.device);
        nk_gemm_destroy(p->chunk_plan);
        cudaStreamDestroy(p->h2d_stream);
        cudaStreamDestroy(p->d2h_stream);
        cudaEventDestroy(p->ev_start);
        cudaEventDestroy(p->ev_done);
        for (int i = 0; i < 12; ++i) cudaEventDestroy(p->ev_up[i]);
        for (int i = 0; i < 32; ++i) cudaEventDestroy(p->ev_g[i]);
    }
    delete p;
    return NK_OK;
}

}  // extern "C"
