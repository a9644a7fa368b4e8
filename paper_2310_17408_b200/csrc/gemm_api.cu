// C ABI of the GEMM library: argument validation, quick returns, the shape selector (tile shape, split-k,
// fast-path eligibility — the role the paper gives to choosing the (mr, nr) micro-kernel and the cache
// parameters per problem, Sections I and IV) and dispatch to the kernels.
#include <algorithm>
#include <atomic>
#include <mutex>
#include <new>
#include <vector>

#include "internal.cuh"

namespace b200gemm {

__device__ uint32_t g_device_status;   // written by bounded waits that expire

constexpr int MAX_DEVICES = 64;
constexpr int64_t DIRECT_MAX_MN = 256 * 256, DIRECT_MAX_K = 384;

// one registered workspace: stream == nullptr is the entry that serves every stream without one of its own
struct Workspace {
    cudaStream_t stream;
    void* ptr;
    size_t bytes;
};

struct DeviceState {
    bool init = false;
    bool arch_ok = false;
    int sms = 0;
    uint32_t* status = nullptr;
    std::vector<Workspace> ws;       // guarded by g_mutex
};

static DeviceState g_dev[MAX_DEVICES];
static std::mutex g_mutex;
static thread_local gemm_config_t t_last_cfg = {};
static thread_local int t_last_cuda_error = 0;
// forcing knobs (tests, benchmarks): per host thread, so that a thread that forces a configuration does not change
// what concurrent callers on other threads get
static thread_local int g_force_kernel = GEMM_KERNEL_AUTO;
static thread_local int g_force_tile_m = 0, g_force_tile_n = 0, g_force_split = 0;
static thread_local bool g_no_tail_split = false;   // gemm_force_tile(.., split_k = 1) also switches the tail split off
static thread_local int g_force_reduction = 0;      // 0 = choose, 1 = separate reduction pass, 2 = inside the kernel (cluster)
static std::atomic<uint32_t> g_last_detail{0};

// the workspace a call on `stream` may use: the one registered for that stream, else the stream-less one
static void workspace_for(DeviceState* st, cudaStream_t stream, void** ws, size_t* bytes) {
    std::lock_guard<std::mutex> lock(g_mutex);
    *ws = nullptr;
    *bytes = 0;
    for (int pass = 0; pass < 2; ++pass)
        for (const Workspace& w : st->ws)
            if (w.stream == (pass == 0 ? stream : nullptr)) {
                *ws = w.ptr;
                *bytes = w.bytes;
                return;
            }
}

static DeviceState* device_state() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& s = g_dev[dev];
    if (!s.init) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return nullptr;
        s.arch_ok = (prop.major == 10);
        s.sms = prop.multiProcessorCount;
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
        s.status = static_cast<uint32_t*>(p);
        s.init = true;
    }
    return &s;
}

int sm_count() {
    DeviceState* s = device_state();
    return (s && s->sms > 0) ? s->sms : 148;
}

bool device_info(uint32_t** status, bool* arch_ok) {
    DeviceState* s = device_state();
    if (!s) return false;
    *status = s->status;
    *arch_ok = s->arch_ok;
    return true;
}

static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }

// ---------------------------------------------------------------- selector

struct Plan {
    int kernel;        // GEMM_KERNEL_*
    int tile;          // SIMT fast: tile id 0..3; tensor: tile_n
    bool pair;         // tensor: 256 x 256 tiles on CTA pairs
    KSplit ks;
    bool repack_a, repack_b;
    int64_t lda_p, ldb_p;     // leading dimensions of the repacked operands
    size_t ws_partials;       // bytes
    size_t ws_total;
    bool cluster_reduce;           // fp32 split-k finished inside the kernel by a thread-block cluster (no workspace)
    int tail_first, tail_splits;   // fp32 tail split (tail_splits <= 1: off)
    int64_t tail_chunk;
};

// k partition: `want` splits of a multiple of `quantum`, no empty split
static KSplit make_split(int64_t k, int want, int quantum) {
    KSplit ks{1, round_up(k > 0 ? k : 1, quantum)};
    if (want <= 1) return ks;
    int64_t chunk = round_up(ceil_div(k, want), quantum);
    int splits = (int)ceil_div(k, chunk);
    if (splits <= 1) return ks;
    ks.splits = splits;
    ks.chunk = chunk;
    return ks;
}

static const int kSimtTileM[4] = {128, 128, 64, 64};
static const int kSimtTileN[4] = {128, 64, 128, 64};

// fp32: pick the CTA tile that fills the SMs best, then split k when the tile count is far below one wave
static void plan_simt(const GemmArgs& a, int sms, size_t ws_avail, Plan* p) {
    p->kernel = GEMM_KERNEL_SIMT_FAST;
    // k worth splitting over CTAs: a cluster sums the ranges inside the kernel, which makes two ranges of 128 pay;
    // the index-map kernel of the convolution layers has no cluster form and needs the reduction pass
    const int64_t k_min_split = a.conv ? 512 : 256;
    const double ctas_per_sm[4] = {2, 3, 3, 6};
    const double eff[4] = {1.0, 0.92, 0.92, 0.80};     // relative math efficiency of the smaller tiles
    int best = 0;
    double best_score = -1;
    for (int t = 0; t < 4; ++t) {
        if (g_force_tile_m && g_force_tile_n && (kSimtTileM[t] != g_force_tile_m || kSimtTileN[t] != g_force_tile_n)) continue;
        const int64_t tm = ceil_div(a.m, kSimtTileM[t]), tn = ceil_div(a.n, kSimtTileN[t]);
        const double tiles = (double)tm * tn;
        const double slots = sms * ctas_per_sm[t];
        const double waves = tiles / slots;
        double full = (double)ceil_div((int64_t)tiles, (int64_t)slots);
        {   // a partly filled last wave that can be cut along k (see the tail split below) costs 1 / splits of a wave
            const int64_t r = (int64_t)tiles % (int64_t)slots;
            int64_t sp = r > 0 ? (int64_t)slots / r : 1;
            if (sp > a.k / 256) sp = a.k / 256;
            if (sp > 8) sp = 8;
            if (tiles > slots && r > 0 && 2 * r <= (int64_t)slots && sp >= 2 && g_force_split == 0 && !g_no_tail_split &&
                (size_t)(r * sp) * kSimtTileM[t] * kSimtTileN[t] * sizeof(float) <= ws_avail)
                full = full - 1.0 + 1.0 / (double)sp;
        }
        double util = waves / full;                                                 // tail effect
        if (tiles * 2 <= slots && a.k >= k_min_split && g_force_split <= 1) {
            // fewer tiles than half the slots: k will be split (below), so what counts is how full the machine is then
            const double smax = std::min(64.0, (double)(a.k / 128));
            util = std::min(1.0, tiles * std::max(1.0, std::floor(std::min(smax, slots / tiles))) / slots);
            // with short k ranges per CTA the narrower tiles (three CTAs per SM) hide latency better than 128 x 128
            // (measured 2-5 % on 1024^3 and 512 x 1568 x 2048)
            static const double eff_split[4] = {0.95, 1.0, 1.0, 0.97};
            util *= eff_split[t] / eff[t];
        }
        const double useful = ((double)a.m * a.n) / (tiles * kSimtTileM[t] * kSimtTileN[t]);   // edge waste
        const double score = util * useful * eff[t];
        if (score > best_score) { best_score = score; best = t; }
    }
    p->tile = best;
    const int64_t tiles = ceil_div(a.m, kSimtTileM[best]) * ceil_div(a.n, kSimtTileN[best]);
    const int64_t slots = (int64_t)(sms * ctas_per_sm[best]);
    int want = 1;
    if (g_force_split > 0) want = g_force_split;
    else if (tiles * 2 <= slots && a.k >= k_min_split) {
        want = (int)(slots / tiles);
        const int64_t max_by_k = a.k / 128;             // keep at least 128 of k per split (measured on 512^3: 2 splits 20.6 us, 4 splits 14.4 us)
        if (want > max_by_k) want = (int)max_by_k;
        if (want > 64) want = 64;
    }
    if (g_force_reduction == 2 && want > CLUSTER_REDUCE_MAX_SPLITS) want = CLUSTER_REDUCE_MAX_SPLITS;
    p->ks = make_split(a.k, want, 16);
    // Up to 8 k ranges per tile are summed inside the kernel by a thread-block cluster (no workspace).  More ranges,
    // or the 128 x 128 tile, keep their partial sums in the workspace and a reduction pass follows; without room
    // for them a wish for more than 8 ranges is cut to 8, which the cluster can do.
    auto clusterable = [&]() { return p->ks.splits > 1 && p->ks.splits <= CLUSTER_REDUCE_MAX_SPLITS && simt_fast_can_cluster_reduce(best) && !a.conv; };
    p->cluster_reduce = g_force_reduction != 1 && clusterable();
    p->ws_partials = (p->ks.splits > 1 && !p->cluster_reduce) ? (size_t)p->ks.splits * a.m * a.n * sizeof(float) : 0;
    if (p->ws_partials > ws_avail) {
        if (g_force_split > 0 && g_force_reduction == 1) { p->kernel = -1; return; }
        p->ks = make_split(a.k, g_force_reduction == 1 ? 1 : std::min(want, CLUSTER_REDUCE_MAX_SPLITS), 16);
        p->cluster_reduce = g_force_reduction != 1 && clusterable();
        if (!p->cluster_reduce) p->ks = make_split(a.k, 1, 16);
        p->ws_partials = 0;
    }
    p->ws_total = p->ws_partials;

    // Tail split: with more tiles than CTA slots the last wave is only partly filled.  Its r tiles are cut into
    // floor(slots / r) k ranges each, so that the last wave fills the machine and takes 1 / splits of a full one;
    // a reduction over those tiles only (tile-local fp32 slots in the workspace) finishes them.
    p->tail_splits = 1;
    p->tail_first = 0x7FFFFFFF;
    if (p->ks.splits == 1 && g_force_split == 0 && !g_no_tail_split && tiles > slots) {
        const int64_t r = tiles % slots;
        if (r > 0 && 2 * r <= slots) {
            int64_t s = slots / r;
            if (s > a.k / 256) s = a.k / 256;
            if (s > 8) s = 8;
            const size_t need = (size_t)(r * s) * kSimtTileM[best] * kSimtTileN[best] * sizeof(float);
            if (s >= 2 && need <= ws_avail) {
                p->tail_first = (int)(tiles - r);
                p->tail_splits = (int)s;
                p->tail_chunk = round_up(ceil_div(a.k, s), 16);
                p->tail_splits = (int)ceil_div(a.k, p->tail_chunk);
                p->ws_partials = (size_t)(r * p->tail_splits) * kSimtTileM[best] * kSimtTileN[best] * sizeof(float);
                p->ws_total = p->ws_partials;
                if (p->tail_splits < 2) { p->tail_splits = 1; p->tail_first = 0x7FFFFFFF; p->ws_partials = p->ws_total = 0; }
            }
        }
    }
}

static void plan_tensor(const GemmArgs& a, int sms, size_t ws_avail, bool a_ok, bool b_ok, Plan* p) {
    p->kernel = GEMM_KERNEL_TENSOR;
    p->repack_a = !a_ok;
    p->repack_b = !b_ok;
    const int64_t a_rows = a.ta ? a.k : a.m, a_cols = a.ta ? a.m : a.k;
    const int64_t b_rows = a.tb ? a.n : a.k, b_cols = a.tb ? a.k : a.n;
    p->lda_p = round_up(a_rows > 0 ? a_rows : 1, 8);
    p->ldb_p = round_up(b_rows > 0 ? b_rows : 1, 8);
    size_t ws_repack = 0;
    if (p->repack_a) ws_repack += (size_t)round_up(p->lda_p * a_cols * 2, 256);
    if (p->repack_b) ws_repack += (size_t)round_up(p->ldb_p * b_cols * 2, 256);
    if (ws_repack > ws_avail) { p->kernel = GEMM_KERNEL_SIMT_GENERIC; return; }

    // Tile width and split-k by a small cost model (microseconds) with constants measured on B200:
    //   - a kernel costs ~7 us before any tile work shows (launch, TMEM/barrier set-up, first loads, last stores)
    //   - one 64-wide k block takes max(tensor time 0.27 us * bn/256, stage bytes / 146 GB/s per-SM fill rate)
    //   - all SMs together fill shared memory from L2 at ~10 TB/s; HBM moves 6.5 TB/s
    //   - the epilogue moves 32 columns of a tile in ~0.45 us
    //   - splitting k adds a reduction pass: ~4 us + (splits + 1) * m * n * 4 bytes at ~5 TB/s
    //   - or, for up to 8 k ranges, the ranges of a tile run as a thread-block cluster and sum the tile through
    //     distributed shared memory: ~2.5 us, no partial sums in memory, but one tile per CTA (no persistent loop), so
    //     only while all CTAs fit the GPU at once (measured: 512 x 1568 x 4608 on 28 tiles of 128 x 256, 4 ranges = 112
    //     CTAs 17.0 us, 6 ranges = 168 CTAs 28.1 us; one launch with a reduction pass 18.9; unsplit 31.0)
    auto cost_us = [&](int bn, int splits, bool cluster) {
        const double tiles = (double)ceil_div(a.m, 128) * (double)ceil_div(a.n, bn);
        const double items = tiles * splits;
        const double rounds = (double)ceil_div((int64_t)items, sms);
        const double kb = (double)ceil_div(ceil_div(a.k, splits), 64);
        const double stage = (128.0 + bn) * 128.0;
        const double t_kb = std::max(0.27 * bn / 256.0, stage / 146e3);
        const double main_us = rounds * kb * t_kb + rounds * (bn / 32) * 0.45;
        const double fill_us = items * kb * stage / 1e7;
        const double mn = (double)a.m * (double)a.n;
        const double hbm_us = (2.0 * ((double)a.m * a.k + (double)a.k * a.n) + 4.0 * mn * (cluster ? 1 : splits)) / 6.5e6;
        double t = 7.0 + std::max(main_us, std::max(fill_us, hbm_us));
        if (splits > 1) t += cluster ? 2.5 : 4.0 + (splits + 1) * mn * 4.0 / 5e6;
        return t;
    };
    int bn = 256, want = 1;
    bool want_cluster = false;
    {
        const int bn_lo = (g_force_tile_n == 64 || g_force_tile_n == 128 || g_force_tile_n == 256) ? g_force_tile_n
                          : (a.n <= 64 ? 64 : 128);
        const int bn_hi = (g_force_tile_n == 64 || g_force_tile_n == 128 || g_force_tile_n == 256) ? g_force_tile_n
                          : (a.n <= 64 ? 64 : (a.n <= 128 ? 128 : 256));
        const int split_opts[] = {1, 2, 3, 4, 6, 8};
        double best = 1e300;
        for (int cand = bn_lo; cand <= bn_hi; cand *= 2)
            for (int so : split_opts)
                for (int cl = 0; cl < 2; ++cl) {
                    if (g_force_split > 0 && so != 1) continue;
                    if (a.acc16 && so != 1) continue;      // a binary16 accumulator is never split along k
                    const int sp = (g_force_split > 0 && !a.acc16) ? g_force_split : so;
                    const bool cluster = cl == 1;
                    if (cluster && (sp < 2 || sp > 8 || g_force_reduction == 1)) continue;
                    if (cluster && g_force_split == 0 && ceil_div(a.m, 128) * ceil_div(a.n, cand) * sp > sms) continue;
                    if (!cluster && sp > 1 && g_force_reduction == 2 && sp <= 8) continue;
                    if (sp > 1 && g_force_split == 0 && a.k / sp < 256) continue;
                    if (sp > 1 && !cluster && ws_repack + (size_t)sp * a.m * a.n * sizeof(float) > ws_avail) {
                        if (g_force_split == 0) continue;
                    }
                    const double c = cost_us(cand, sp, cluster);
                    if (c < best) { best = c; bn = cand; want = sp; want_cluster = cluster; }
                }
    }
    p->tile = bn;
    // CTA pairs (256 x 256 tiles) fill a third less shared memory per flop, which is what limits the 128 x 256
    // kernel: measured 9 % faster main loops (4096^3, 8192^3, the large VGG16 shapes), but ~2.5 us more fixed
    // cost per launch (cluster set-up, cross-CTA barriers).  Taken when every pair has work and the main loops
    // of the 128 x 256 kernel would run for 10 us or more (measured: ahead from ~14 us on, behind at ~4 us).
    {
        const int64_t pair_tiles = ceil_div(a.m, 256) * ceil_div(a.n, 256);
        const double rounds = (double)ceil_div(ceil_div(a.m, 128) * ceil_div(a.n, 256), sms);
        const double main_us = rounds * (double)ceil_div(a.k, 64) * 0.27;
        p->pair = bn == 256 && want == 1 && a.m > 128 && pair_tiles >= sms / 2 && main_us >= 10.0;
        if (want_cluster) p->pair = false;
    }
    if (g_force_tile_m == 256) p->pair = bn == 256;
    if (g_force_tile_m == 128 || a.acc16) p->pair = false;      // the binary16 accumulator exists in the single-CTA kernel only
    p->ks = make_split(a.k, want, 64);
    p->cluster_reduce = want_cluster && !p->pair && p->ks.splits >= 2 && p->ks.splits <= 8;      // single-CTA kernel only
    p->ws_partials = (p->ks.splits > 1 && !p->cluster_reduce) ? (size_t)p->ks.splits * a.m * a.n * sizeof(float) : 0;
    if (ws_repack + p->ws_partials > ws_avail) {
        if (g_force_split > 0) { p->kernel = -1; return; }
        p->ks = make_split(a.k, 1, 64);
        p->ws_partials = 0;
    }
    p->tail_splits = 1;
    p->tail_first = 0x7FFFFFFF;
    p->ws_total = ws_repack + p->ws_partials;
}

// Problems this small are a few microseconds of work however they are run; what counts is the length of the
// longest dependency chain, and the kernel without staging (no shared memory, no barriers, 16 entries of C per
// thread) has the shortest one.  Thresholds measured on B200 against the staged kernel.
static bool direct_preferred(int64_t m, int64_t n, int64_t k) {
    // measured (graph replay, one problem): ahead of the staged kernel up to 256^3 (14 us against 16) and by 1.3-2x
    // below 128^3; behind once k is long enough for the staged kernel to split it (128 x 128 x 512: 26 us against 10)
    return (m * n <= 128 * 128 && k <= DIRECT_MAX_K) || (m * n <= DIRECT_MAX_MN && k <= 256);
}

static Plan make_plan(const GemmArgs& a, int sms, size_t ws_avail) {
    Plan p{};
    p.ks = KSplit{1, a.k > 0 ? a.k : 1};
    int forced = g_force_kernel;
    if (forced == GEMM_KERNEL_SIMT_GENERIC && !a.conv) { p.kernel = GEMM_KERNEL_SIMT_GENERIC; return p; }
    if (a.dtype == GEMM_F32) {
        if (!a.conv && (forced == GEMM_KERNEL_SIMT_DIRECT || (forced == GEMM_KERNEL_AUTO && direct_preferred(a.m, a.n, a.k) &&
                                                               g_force_tile_m == 0 && g_force_split == 0))) {
            p.kernel = GEMM_KERNEL_SIMT_DIRECT;
            return p;
        }
        plan_simt(a, sms, ws_avail, &p);
        return p;
    }
    // 16-bit inputs: tensor path if the operands are (or can be made) addressable by TMA
    auto aligned = [](const void* ptr, int64_t ld) { return (reinterpret_cast<uintptr_t>(ptr) & 15) == 0 && ld % 8 == 0; };
    GemmArgs probe = a;
    // a lowered convolution operand is fetched by TMA from the activation tensor: nothing of B to align or repack
    const bool a_ok = aligned(a.A, a.lda), b_ok = a.conv ? true : aligned(a.B, a.ldb);
    if (a.conv) { probe.B = nullptr; probe.ldb = 8; }
    if (!a_ok) { probe.A = nullptr; probe.lda = 8; }      // judged on the repacked layout
    if (!b_ok) { probe.B = nullptr; probe.ldb = 8; }
    if (!tensor_eligible(probe)) { p.kernel = GEMM_KERNEL_SIMT_GENERIC; return p; }
    plan_tensor(a, sms, ws_avail, a_ok, b_ok, &p);
    return p;
}

// ---------------------------------------------------------------- validation

static int validate(int dtype, char ta, char tb, int64_t m, int64_t n, int64_t k, float alpha, const void* A,
                    int64_t lda, const void* B, int64_t ldb, const void* C, int64_t ldc, bool* tA, bool* tB) {
    auto tr = [](char c, bool* t) {
        switch (c) {
            case 'N': case 'n': *t = false; return true;
            case 'T': case 't': case 'C': case 'c': *t = true; return true;
            default: return false;
        }
    };
    if (dtype != GEMM_F32 && dtype != GEMM_F16 && dtype != GEMM_BF16 && dtype != GEMM_F16_C16 && dtype != GEMM_BF16_C16 &&
        dtype != GEMM_F32_TC && dtype != GEMM_F16_ACC16)
        return -1;
    if (!tr(ta, tA)) return -2;
    if (!tr(tb, tB)) return -3;
    if (m < 0) return -4;
    if (n < 0) return -5;
    if (k < 0) return -6;
    const int64_t a_rows = *tA ? k : m, b_rows = *tB ? n : k;
    const bool needs_ab = m > 0 && n > 0 && k > 0 && alpha != 0.0f;
    const int es = elem_size(dtype);
    if (needs_ab && A == nullptr) return -8;
    if (A != nullptr && (reinterpret_cast<uintptr_t>(A) % es) != 0) return -8;
    if (lda < (a_rows > 1 ? a_rows : 1)) return -9;
    if (needs_ab && B == nullptr) return -10;
    if (B != nullptr && (reinterpret_cast<uintptr_t>(B) % es) != 0) return -10;
    if (ldb < (b_rows > 1 ? b_rows : 1)) return -11;
    if (m > 0 && n > 0 && C == nullptr) return -13;
    if (C != nullptr && (reinterpret_cast<uintptr_t>(C) % c_elem_size(dtype)) != 0) return -13;
    if (ldc < (m > 1 ? m : 1)) return -14;
    return 0;
}

static int fail_launch(cudaError_t e) {
    t_last_cuda_error = (int)e;
    return GEMM_ERR_LAUNCH;
}

static int run_gemm(const GemmArgs& a0, DeviceState* st, size_t ws_skip = 0);

// ---------------------------------------------------------------- fp32 on the tensor cores (GEMM_F32_TC)

// Workspace for the bfloat16 pieces of A and B: three copies each, leading dimension rounded up to 8 elements.
struct Split3Layout {
    int64_t a_rows, a_cols, b_rows, b_cols, lda_p, ldb_p;
    size_t a_piece, b_piece, total;      // bytes: three separate pieces per operand (six products, six launches)
    // the pieces of an operand one after the other along k, k padded with zeros to a multiple of 64 (one launch)
    int64_t seg_k, lda_f, ldb_f;
    size_t a_fused, b_fused, a_step, b_step, total_fused;      // bytes; *_step = distance between two pieces
};
static Split3Layout split3_layout(const GemmArgs& a) {
    Split3Layout L;
    L.a_rows = a.ta ? a.k : a.m; L.a_cols = a.ta ? a.m : a.k;
    L.b_rows = a.tb ? a.n : a.k; L.b_cols = a.tb ? a.k : a.n;
    L.lda_p = round_up(L.a_rows, 8);
    L.ldb_p = round_up(L.b_rows, 8);
    L.a_piece = (size_t)round_up(L.lda_p * L.a_cols * 2, 256);
    L.b_piece = (size_t)round_up(L.ldb_p * L.b_cols * 2, 256);
    L.total = 3 * (L.a_piece + L.b_piece);
    L.seg_k = round_up(a.k, 64);
    // k is the row index of a stored operand (A^T, B): pieces stacked in the rows, one leading dimension of 3 * seg_k;
    // k is the column index (A, B^T): pieces are runs of seg_k columns
    L.lda_f = a.ta ? 3 * L.seg_k : L.lda_p;
    L.ldb_f = a.tb ? L.ldb_p : 3 * L.seg_k;
    L.a_step = a.ta ? (size_t)L.seg_k * 2 : (size_t)L.lda_p * L.seg_k * 2;
    L.b_step = a.tb ? (size_t)L.ldb_p * L.seg_k * 2 : (size_t)L.seg_k * 2;
    L.a_fused = (size_t)round_up(a.ta ? 3 * L.seg_k * a.m * 2 : L.lda_p * 3 * L.seg_k * 2, 256);
    L.b_fused = (size_t)round_up(a.tb ? L.ldb_p * 3 * L.seg_k * 2 : 3 * L.seg_k * a.n * 2, 256);
    L.total_fused = L.a_fused + L.b_fused;
    return L;
}
// worth it from about here on.  As one launch on CTA pairs (at least 16 tiles of 256 x 256), measured against the exact
// kernel: 1024^3 51 against 53 us, 1280^3 64 against 91, 1536^3 74 against 140, 2048^3 99 against 309 us, 8192^3 5.5
// against 18.4 ms.  As six launches (fewer tiles): 1024^3 83 against 57 us, 2048^3 153 against 326.
static bool split3_one_launch_shape(const GemmArgs& a) {
    return a.m > 128 && ceil_div(a.m, 256) * ceil_div(a.n, 256) >= 16;
}
static bool split3_worthwhile(const GemmArgs& a) {
    const double volume = (double)a.m * (double)a.n * (double)a.k;
    const double from = split3_one_launch_shape(a) ? 1280.0 : 1536.0;
    return volume >= from * from * from && a.m >= 128 && a.n >= 128 && a.k >= 64;
}

// The six piece products as ONE multiplication on CTA pairs: op(A) and op(B) hold their pieces one after the other along
// k and every tile's k loop walks the six (piece of A, piece of B) segments, smallest products first, into one fp32
// accumulator in TMEM; alpha and beta are applied once, in the epilogue.  For problems whose 256 x 256 tiles give
// every CTA pair work.
static bool split3_fused_fits(const GemmArgs& a, const Split3Layout& L, int sms, size_t ws_bytes) {
    if (ws_bytes < L.total_fused || g_force_tile_m == 128 || g_force_tile_n == 128 || g_force_tile_n == 64) return false;
    if (3 * L.seg_k > 0x7FFFFFFFLL) return false;
    return split3_one_launch_shape(a);      // one k loop is six ordinary ones long: a tile per pair is not needed
}
static int run_f32_split3_fused(const GemmArgs& a, const Split3Layout& L, void* ws) {
    uint8_t* pa = static_cast<uint8_t*>(ws);
    uint8_t* pb = pa + L.a_fused;
    // k runs along the rows of a stored A^T / B and along the columns of a stored A / B^T
    cudaError_t e = a.ta ? launch_split3(static_cast<const float*>(a.A), L.a_rows, L.a_cols, a.lda, pa, pa + L.a_step, pa + 2 * L.a_step,
                                         L.lda_f, a.stream, L.seg_k, 0)
                         : launch_split3(static_cast<const float*>(a.A), L.a_rows, L.a_cols, a.lda, pa, pa + L.a_step, pa + 2 * L.a_step,
                                         L.lda_f, a.stream, 0, L.seg_k);
    if (e == cudaSuccess)
        e = a.tb ? launch_split3(static_cast<const float*>(a.B), L.b_rows, L.b_cols, a.ldb, pb, pb + L.b_step, pb + 2 * L.b_step,
                                 L.ldb_f, a.stream, 0, L.seg_k)
                 : launch_split3(static_cast<const float*>(a.B), L.b_rows, L.b_cols, a.ldb, pb, pb + L.b_step, pb + 2 * L.b_step,
                                 L.ldb_f, a.stream, L.seg_k, 0);
    if (e != cudaSuccess) return fail_launch(e);
    GemmArgs g = a;
    g.dtype = GEMM_BF16;
    g.split3 = 0;
    g.A = pa; g.lda = L.lda_f;
    g.B = pb; g.ldb = L.ldb_f;
    g.k = 3 * L.seg_k;          // the extent of the stored operands along k
    g.seg_k = L.seg_k;
    gemm_config_t cfg{};
    e = launch_tensor_pair(g, KSplit{1, g.k}, nullptr, &cfg);
    if (e != cudaSuccess) return fail_launch(e);
    cfg.launches = 3;
    note_config(cfg);
    return GEMM_OK;
}

// C <- alpha * sum of the six piece products + beta*C: six bfloat16 GEMMs accumulating into C, smallest terms first
static int run_f32_split3(const GemmArgs& a, DeviceState* st, void* ws, size_t ws_bytes) {
    const Split3Layout L = split3_layout(a);
    if (split3_fused_fits(a, L, st->sms, ws_bytes)) return run_f32_split3_fused(a, L, ws);
    uint8_t* base = static_cast<uint8_t*>(ws);
    void* ap[3] = {base, base + L.a_piece, base + 2 * L.a_piece};
    void* bp[3] = {base + 3 * L.a_piece, base + 3 * L.a_piece + L.b_piece, base + 3 * L.a_piece + 2 * L.b_piece};
    cudaError_t e = launch_split3(static_cast<const float*>(a.A), L.a_rows, L.a_cols, a.lda, ap[0], ap[1], ap[2], L.lda_p, a.stream);
    if (e == cudaSuccess)
        e = launch_split3(static_cast<const float*>(a.B), L.b_rows, L.b_cols, a.ldb, bp[0], bp[1], bp[2], L.ldb_p, a.stream);
    if (e != cudaSuccess) return fail_launch(e);
    static const int order[6][2] = {{2, 0}, {0, 2}, {1, 1}, {1, 0}, {0, 1}, {0, 0}};      // (piece of A, piece of B)
    int launches = 2;
    gemm_config_t last{};
    for (int t = 0; t < 6; ++t) {
        GemmArgs g = a;
        g.dtype = GEMM_BF16;
        g.split3 = 0;
        g.A = ap[order[t][0]]; g.lda = L.lda_p;
        g.B = bp[order[t][1]]; g.ldb = L.ldb_p;
        if (t > 0) g.beta = 1.0f;               // later products accumulate onto the earlier ones
        const int rc = run_gemm(g, st, L.total + (size_t)0);
        if (rc != GEMM_OK) return rc;
        launches += t_last_cfg.launches;
        last = t_last_cfg;
    }
    last.launches = launches;
    t_last_cfg = last;
    (void)ws_bytes;
    return GEMM_OK;
}

static int run_gemm(const GemmArgs& a0, DeviceState* st, size_t ws_skip) {
    GemmArgs a = a0;
    gemm_config_t cfg{};
    cfg.split_k = 1;
    cfg.launches = 1;
    cudaError_t e;

    if (a.alpha == 0.0f || a.k == 0) {
        cfg.kernel = GEMM_KERNEL_SCALE_ONLY;
        if (a.beta == 1.0f) { cfg.launches = 0; t_last_cfg = cfg; return GEMM_OK; }
        e = launch_scale(a);
        t_last_cfg = cfg;
        return e == cudaSuccess ? GEMM_OK : fail_launch(e);
    }

    if (a.split3 && a.dtype == GEMM_F32 && !a.conv && ws_skip == 0 && g_force_kernel != GEMM_KERNEL_SIMT_FAST &&
        g_force_kernel != GEMM_KERNEL_SIMT_GENERIC && g_force_kernel != GEMM_KERNEL_SIMT_DIRECT &&
        (split3_worthwhile(a) || g_force_kernel == GEMM_KERNEL_TENSOR) &&
        a.m <= 0x7FFFFFFFLL && a.n <= 0x7FFFFFFFLL && a.k <= 0x7FFFFFFFLL) {
        void* ws3;
        size_t ws3_bytes;
        workspace_for(st, a.stream, &ws3, &ws3_bytes);
        const Split3Layout L3 = split3_layout(a);
        if (ws3 != nullptr && (ws3_bytes >= L3.total || split3_fused_fits(a, L3, st->sms, ws3_bytes)))
            return run_f32_split3(a, st, ws3, ws3_bytes);
    }
    a.split3 = 0;      // from here on: the exact fp32 path

    void* ws;
    size_t ws_bytes;
    workspace_for(st, a.stream, &ws, &ws_bytes);
    if (ws_skip > 0) {      // the head of the workspace is in use by the caller (a lowered activation matrix)
        if (ws == nullptr || ws_bytes < ws_skip) return GEMM_ERR_WORKSPACE;
        ws = static_cast<uint8_t*>(ws) + ws_skip;
        ws_bytes -= ws_skip;
    }
    // 16-bit inputs with at most 64 rows of C and many columns (the C_out = 64 layers): a 128-row MMA would run half
    // empty and only half of the epilogue warps would have rows to store.  Exchange the roles of the operands instead:
    // C^T = op(B)^T op(A)^T, the columns of C (pixels) become the 128 rows of the MMA, its 64 rows the MMA's N, and a
    // lane of the epilogue writes consecutive floats of its column of C.
    if (a.dtype != GEMM_F32 && !a.conv && !a.out16 && !a.acc16 && a.m <= 64 && a.n >= 1024 && g_force_tile_m == 0 &&
        g_force_tile_n == 0 && g_force_split == 0 && g_force_kernel != GEMM_KERNEL_SIMT_GENERIC) {
        GemmArgs x = a;
        x.m = a.n; x.n = a.m;
        x.A = a.B; x.lda = a.ldb; x.ta = !a.tb;
        x.B = a.A; x.ldb = a.lda; x.tb = !a.ta;
        x.ct = 1;
        Plan px = make_plan(x, st->sms, ws_bytes);
        if (px.kernel == GEMM_KERNEL_TENSOR && px.tile == 64 && px.ks.splits == 1 && !px.pair) {
            uint8_t* w = static_cast<uint8_t*>(ws);
            if (px.repack_a) {
                const int64_t rows = x.ta ? x.k : x.m, cols = x.ta ? x.m : x.k;
                e = launch_repack16(x.A, rows, cols, x.lda, w, px.lda_p, x.stream);
                if (e != cudaSuccess) return fail_launch(e);
                x.A = w; x.lda = px.lda_p;
                w += round_up(px.lda_p * cols * 2, 256);
                cfg.repacked |= 2; cfg.launches++;      // (the caller's B)
            }
            if (px.repack_b) {
                const int64_t rows = x.tb ? x.n : x.k, cols = x.tb ? x.k : x.n;
                e = launch_repack16(x.B, rows, cols, x.ldb, w, px.ldb_p, x.stream);
                if (e != cudaSuccess) return fail_launch(e);
                x.B = w; x.ldb = px.ldb_p;
                cfg.repacked |= 1; cfg.launches++;      // (the caller's A)
            }
            e = launch_tensor(x, 64, px.ks, nullptr, &cfg, false);
            std::swap(cfg.tile_m, cfg.tile_n);           // reported in the caller's orientation
            t_last_cfg = cfg;
            return e == cudaSuccess ? GEMM_OK : fail_launch(e);
        }
    }
    Plan p = make_plan(a, st->sms, ws_bytes);
    if (p.kernel < 0) return GEMM_ERR_WORKSPACE;

    if (p.kernel == GEMM_KERNEL_SIMT_GENERIC) {
        e = launch_simt_generic(a, &cfg);
        t_last_cfg = cfg;
        return e == cudaSuccess ? GEMM_OK : fail_launch(e);
    }
    if (p.kernel == GEMM_KERNEL_SIMT_DIRECT) {
        e = launch_simt_direct(a, 0, 0, 0, 1, &cfg);
        t_last_cfg = cfg;
        return e == cudaSuccess ? GEMM_OK : fail_launch(e);
    }

    uint8_t* wsp = static_cast<uint8_t*>(ws);
    if (p.kernel == GEMM_KERNEL_TENSOR) {
        if (p.repack_a) {
            const int64_t rows = a.ta ? a.k : a.m, cols = a.ta ? a.m : a.k;
            e = launch_repack16(a.A, rows, cols, a.lda, wsp, p.lda_p, a.stream);
            if (e != cudaSuccess) return fail_launch(e);
            a.A = wsp; a.lda = p.lda_p;
            wsp += round_up(p.lda_p * cols * 2, 256);
            cfg.repacked |= 1; cfg.launches++;
        }
        if (p.repack_b) {
            const int64_t rows = a.tb ? a.n : a.k, cols = a.tb ? a.k : a.n;
            e = launch_repack16(a.B, rows, cols, a.ldb, wsp, p.ldb_p, a.stream);
            if (e != cudaSuccess) return fail_launch(e);
            a.B = wsp; a.ldb = p.ldb_p;
            wsp += round_up(p.ldb_p * cols * 2, 256);
            cfg.repacked |= 2; cfg.launches++;
        }
    }
    float* partials = p.ks.splits > 1 ? reinterpret_cast<float*>(wsp) : nullptr;
    if (p.kernel == GEMM_KERNEL_TENSOR) {
        e = p.pair ? launch_tensor_pair(a, p.ks, partials, &cfg)
                   : launch_tensor(a, p.tile, p.ks, partials, &cfg, p.cluster_reduce);
        if (e != cudaSuccess && p.cluster_reduce) {      // as below for the fp32 kernel: without the cluster, k unsplit
            (void)cudaGetLastError();
            p.cluster_reduce = false;
            p.ks = make_split(a.k, 1, 64);
            partials = nullptr;
            e = launch_tensor(a, p.tile, p.ks, nullptr, &cfg, false);
        }
    } else if (p.tail_splits > 1) {
        TailSplit tail{p.tail_first, p.tail_splits, p.tail_chunk, reinterpret_cast<float*>(wsp)};
        e = launch_simt_fast(a, p.tile, p.ks, nullptr, &cfg, tail);
        if (e == cudaSuccess) e = launch_tail_reduce(a, kSimtTileM[p.tile], kSimtTileN[p.tile], SIMT_GROUP, tail);
        cfg.launches++;
        cfg.tail_split = p.tail_splits;
    } else {
        e = launch_simt_fast(a, p.tile, p.ks, partials, &cfg, TailSplit{0x7FFFFFFF, 1, 0, nullptr}, p.cluster_reduce);
        if (e != cudaSuccess && p.cluster_reduce) {
            // the device would not take the cluster (a restricted context, say): the same tile, k unsplit
            (void)cudaGetLastError();
            p.cluster_reduce = false;
            p.ks = make_split(a.k, 1, 16);
            e = launch_simt_fast(a, p.tile, p.ks, nullptr, &cfg);
        }
    }
    if (e == cudaSuccess && p.ks.splits > 1 && !p.cluster_reduce) {
        e = launch_splitk_reduce(a, p.ks.splits, partials);
        cfg.launches++;
    }
    t_last_cfg = cfg;
    return e == cudaSuccess ? GEMM_OK : fail_launch(e);
}

// entry for the convolution front end (conv_api.cu)
int dispatch_gemm(const GemmArgs& a, size_t ws_skip) {
    DeviceState* st = device_state();
    if (!st) return GEMM_ERR_LAUNCH;
    if (!st->arch_ok) return GEMM_ERR_ARCH;
    GemmArgs b = a;
    b.status = st->status;
    return run_gemm(b, st, ws_skip);
}

bool registered_workspace(cudaStream_t stream, void** ws, size_t* bytes) {
    DeviceState* st = device_state();
    if (!st) return false;
    workspace_for(st, stream, ws, bytes);
    return true;
}

void note_lowering(int how) { t_last_cfg.lowering = how; }
void note_launch_error(cudaError_t e) { t_last_cuda_error = (int)e; }
void note_config(const gemm_config_t& cfg) { t_last_cfg = cfg; }

}  // namespace b200gemm

using namespace b200gemm;

extern "C" {

int gemm(int dtype, char transA, char transB, int64_t m, int64_t n, int64_t k, float alpha, const void* A, int64_t lda,
         const void* B, int64_t ldb, float beta, void* C, int64_t ldc, void* stream) {
    bool ta = false, tb = false;
    int bad = validate(dtype, transA, transB, m, n, k, alpha, A, lda, B, ldb, C, ldc, &ta, &tb);
    if (bad) return bad;
    if (m == 0 || n == 0) {
        gemm_config_t cfg{};
        cfg.kernel = GEMM_KERNEL_SCALE_ONLY;
        t_last_cfg = cfg;
        return GEMM_OK;
    }
    DeviceState* st = device_state();
    if (!st) return GEMM_ERR_LAUNCH;
    if (!st->arch_ok) return GEMM_ERR_ARCH;
    GemmArgs a{input_dtype(dtype), ta, tb, m, n, k, alpha, beta, A, B, static_cast<float*>(C), lda, ldb, ldc,
               static_cast<cudaStream_t>(stream), st->status};
    a.out16 = output16(dtype);
    a.split3 = dtype == GEMM_F32_TC ? 1 : 0;
    a.acc16 = dtype == GEMM_F16_ACC16 ? 1 : 0;
    return run_gemm(a, st);
}

int gemm_strided_batched(int dtype, char transA, char transB, int64_t m, int64_t n, int64_t k, float alpha, const void* A,
                         int64_t lda, int64_t strideA, const void* B, int64_t ldb, int64_t strideB, float beta, void* C,
                         int64_t ldc, int64_t strideC, int64_t batch, void* stream) {
    bool ta = false, tb = false;
    // gemm()'s checks, with the positions of this argument list
    static const int pos[16] = {0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 11, 12, 0, 15, 16, 0};
    const int bad = validate(dtype, transA, transB, m, n, k, alpha, A, lda, B, ldb, C, ldc, &ta, &tb);
    if (bad) return -pos[-bad];
    if (strideA < 0) return -10;
    if (strideB < 0) return -13;
    if (strideC < 0) return -17;
    if (batch < 0) return -18;
    if (batch > 1 && m > 0 && n > 0 && strideC < ldc * n) return -17;      // results of different problems would overlap
    gemm_config_t cfg{};
    cfg.kernel = GEMM_KERNEL_SCALE_ONLY;
    cfg.split_k = 1;
    if (m == 0 || n == 0 || batch == 0) { t_last_cfg = cfg; return GEMM_OK; }
    DeviceState* st = device_state();
    if (!st) return GEMM_ERR_LAUNCH;
    if (!st->arch_ok) return GEMM_ERR_ARCH;
    GemmArgs a{input_dtype(dtype), ta, tb, m, n, k, alpha, beta, A, B, static_cast<float*>(C), lda, ldb, ldc,
               static_cast<cudaStream_t>(stream), st->status};
    a.out16 = output16(dtype);
    a.acc16 = dtype == GEMM_F16_ACC16 ? 1 : 0;
    const int es = elem_size(dtype), es_c = c_elem_size(dtype);
    auto at = [&](int64_t b0) {      // the call's arguments moved to problem b0
        GemmArgs x = a;
        if (A) x.A = static_cast<const uint8_t*>(A) + b0 * strideA * es;
        if (B) x.B = static_cast<const uint8_t*>(B) + b0 * strideB * es;
        x.C = reinterpret_cast<float*>(static_cast<uint8_t*>(C) + b0 * strideC * es_c);
        return x;
    };
    constexpr int64_t CHUNK = 65535;      // problems per launch (grid limit of the batch dimension)
    cudaError_t e = cudaSuccess;
    int launches = 0;
    if (alpha == 0.0f || k == 0) {
        if (beta != 1.0f)
            for (int64_t b0 = 0; b0 < batch && e == cudaSuccess; b0 += CHUNK, ++launches)
                e = launch_scale(at(b0), strideC, std::min(CHUNK, batch - b0));
        cfg.launches = launches;
        t_last_cfg = cfg;
        return e == cudaSuccess ? GEMM_OK : fail_launch(e);
    }
    // one launch covers the whole batch when the problems are small: fp32 through the kernel without staging
    // (tiny) or the register-blocked kernel with 64 x 64 or 128 x 128 CTA tiles; 16-bit inputs through the
    // bounds-checked kernel.  Large problems gain nothing from sharing a launch: each goes through gemm().
    const double work = (double)m * (double)n * (double)k;
    const int forced = g_force_kernel;
    if (a.dtype == GEMM_F32 && (work <= 512.0 * 512.0 * 512.0 || forced == GEMM_KERNEL_SIMT_FAST || forced == GEMM_KERNEL_SIMT_DIRECT) &&
        forced != GEMM_KERNEL_SIMT_GENERIC) {
        // A few problems: what counts is the length of one problem's dependency chain, as for a single call.  Many
        // problems: throughput; the kernel without staging tops out near 22 TFLOP/s (every operand element comes
        // through L1 once per thread that uses it), the staged kernel reaches 40-49, but its smallest tile is 64 x 64,
        // so problems up to about 48 x 48 are still better off without staging (measured: 32^3 x 16384 71 us against
        // 149, 64^3 x 4096 107 us against 55).
        const bool direct = forced == GEMM_KERNEL_SIMT_DIRECT ||
                            (forced == GEMM_KERNEL_AUTO && (batch <= 4 ? direct_preferred(m, n, k) : m * n <= 48 * 48));
        auto padded = [&](int64_t t) { return (double)(ceil_div(m, t) * t) * (double)(ceil_div(n, t) * t); };
        const int64_t tiles128 = ceil_div(m, 128) * ceil_div(n, 128);
        // 64 x 64 tiles when they waste less of the padded area (their inner loop is ~20 % behind the 128 x 128 one) or when
        // 128 x 128 tiles would not fill the GPU
        const int tile = (padded(64) * 1.25 < padded(128) || tiles128 * batch < 2 * (int64_t)st->sms) ? 3 : 0;
        if (direct) {      // numbers its work units through the whole batch: one launch however many problems
            e = launch_simt_direct(a, strideA, strideB, strideC, batch, &cfg);
            launches = 1;
        } else {
            for (int64_t b0 = 0; b0 < batch && e == cudaSuccess; b0 += CHUNK, ++launches)
                e = launch_simt_fast_batched(at(b0), tile, strideA, strideB, strideC, std::min(CHUNK, batch - b0), &cfg);
        }
        cfg.launches = launches;
        t_last_cfg = cfg;
        return e == cudaSuccess ? GEMM_OK : fail_launch(e);
    }
    // 16-bit batches on the tensor cores in one launch, when TMA can address the operands of every problem: 16-byte
    // aligned bases, leading dimensions and batch strides (a shared operand, stride 0, is fine)
    if (a.dtype != GEMM_F32 && !a.acc16 && forced != GEMM_KERNEL_SIMT_GENERIC && st->arch_ok && batch > 1 && k > 0 && alpha != 0.0f &&
        g_force_tile_m == 0 && g_force_split == 0 && m <= 0x7FFFFFFFLL && n <= 0x7FFFFFFFLL && k <= 0x7FFFFFFFLL &&
        (reinterpret_cast<uintptr_t>(A) & 15) == 0 && (reinterpret_cast<uintptr_t>(B) & 15) == 0 && lda % 8 == 0 && ldb % 8 == 0 &&
        strideA % 8 == 0 && strideB % 8 == 0 && strideA >= 0 && strideB >= 0 && (double)m * n * batch >= 128.0 * 128.0 * 8.0) {
        const int tile_n = n <= 64 ? 64 : (n <= 128 ? 128 : 256);
        e = launch_tensor_batched(a, tile_n, strideA, strideB, strideC, batch, &cfg);
        if (e == cudaSuccess) {
            cfg.launches = 1;
            t_last_cfg = cfg;
            return GEMM_OK;
        }
        (void)cudaGetLastError();      // a map the driver would not encode: the paths below take the batch
        e = cudaSuccess;
    }
    if (forced == GEMM_KERNEL_SIMT_GENERIC || (a.dtype != GEMM_F32 && work <= 128.0 * 128.0 * 128.0)) {
        for (int64_t b0 = 0; b0 < batch && e == cudaSuccess; b0 += CHUNK, ++launches)
            e = launch_simt_generic(at(b0), &cfg, strideA, strideB, strideC, std::min(CHUNK, batch - b0));
        cfg.launches = launches;
        t_last_cfg = cfg;
        return e == cudaSuccess ? GEMM_OK : fail_launch(e);
    }
    int rc = GEMM_OK;
    for (int64_t b0 = 0; b0 < batch && rc == GEMM_OK; ++b0) {
        rc = run_gemm(at(b0), st);
        launches += t_last_cfg.launches;
    }
    t_last_cfg.launches = launches;
    return rc;
}

// copy a rows x cols window of a column-major matrix (element size es, leading dimension ld on both sides)
static cudaError_t copy_window(void* dst, const void* src, int64_t rows, int64_t cols, int64_t ld, int es,
                               cudaMemcpyKind kind, cudaStream_t s) {
    if (rows == 0 || cols == 0) return cudaSuccess;
    if (rows == ld) return cudaMemcpyAsync(dst, src, (size_t)rows * cols * es, kind, s);
    return cudaMemcpy2DAsync(dst, (size_t)ld * es, src, (size_t)ld * es, (size_t)rows * es, (size_t)cols, kind, s);
}

struct HostPipe {          // per device: what gemm_host keeps between calls
    bool init = false;
    cudaStream_t in = nullptr, out = nullptr;      // the two copy streams
    cudaMemPool_t pool = nullptr;                   // the library's own pool for the staging buffers of A, B and C
    std::vector<cudaEvent_t> events;                // grown on demand, reused by every call
};
static HostPipe g_pipe[MAX_DEVICES];
static std::mutex g_host_mutex;                     // one gemm_host per process at a time (they share the pipe)

// columns per panel of C: a multiple of the CTA tile such that the panel's tiles fill whole waves of the GPU as nearly as
// possible (a panel is one gemm() call), among the widths that cut C into 4 .. 12 panels
static int64_t host_panel_columns(int dtype, int64_t m, int64_t n, int sms, bool wire_bound) {
    const int tile = dtype == GEMM_F32 ? 128 : 256;                 // fp32: 128 x 128 CTA tiles; 16-bit: 256 x 256 on CTA pairs
    const int64_t slots = dtype == GEMM_F32 ? 2 * (int64_t)sms : sms / 2;
    const int64_t tiles_m = ceil_div(m, tile), tiles_n = ceil_div(n, tile);
    int64_t best = tiles_n;
    double best_eff = -1.0;
    for (int64_t c = 1; c <= tiles_n; ++c) {
        const int64_t panels = ceil_div(tiles_n, c);
        if (panels < 4 || panels > 12) continue;
        const int64_t tiles = tiles_m * c;
        // when the transfers set the pace the arithmetic has slack: finer panels (a shorter last step after the last
        // byte has arrived), as long as a panel still gives every SM a tile
        if (wire_bound && panels < 6 && tiles_m * ceil_div(tiles_n, 6) * 2 >= slots) continue;
        const double eff = (double)tiles / (double)(ceil_div(tiles, slots) * slots);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = c; }
    }
    return best * tile;
}

int gemm_host(int dtype, char transA, char transB, int64_t m, int64_t n, int64_t k, float alpha, const void* A_host,
              int64_t lda, const void* B_host, int64_t ldb, float beta, void* C_host, int64_t ldc, void* stream) {
    bool ta = false, tb = false;
    int bad = validate(dtype, transA, transB, m, n, k, alpha, A_host, lda, B_host, ldb, C_host, ldc, &ta, &tb);
    if (bad) return bad;
    if (m == 0 || n == 0) return GEMM_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return GEMM_ERR_LAUNCH;
    DeviceState* st = device_state();
    if (!st) return GEMM_ERR_LAUNCH;
    std::lock_guard<std::mutex> host_lock(g_host_mutex);
    HostPipe* pipe = &g_pipe[dev];
    if (!pipe->init) {
        // a pool of the library's own, so that keeping freed staging buffers for the next call changes nothing for
        // the application's default pool
        cudaMemPoolProps props = {};
        props.allocType = cudaMemAllocationTypePinned;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = dev;
        if (cudaMemPoolCreate(&pipe->pool, &props) != cudaSuccess) return fail_launch(cudaGetLastError());
        uint64_t keep = ~0ull;
        cudaMemPoolSetAttribute(pipe->pool, cudaMemPoolAttrReleaseThreshold, &keep);
        if (cudaStreamCreateWithFlags(&pipe->in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&pipe->out, cudaStreamNonBlocking) != cudaSuccess)
            return fail_launch(cudaGetLastError());
        pipe->init = true;
    }
    const int es = elem_size(dtype);       // of A and B
    const bool needs_ab = (k > 0 && alpha != 0.0f);
    const int64_t a_rows = ta ? k : m, a_cols = ta ? m : k;
    const size_t a_bytes = needs_ab ? (size_t)lda * a_cols * es : 0;
    const size_t b_bytes = needs_ab ? (size_t)ldb * (tb ? k : n) * es : 0;
    const int es_c = c_elem_size(dtype);
    const size_t c_bytes = (size_t)ldc * n * es_c;

    // Column panels of C (and of op(B)) flow through a three-stream pipeline: panel p+1 is copied in while panel p
    // is multiplied and panel p-1 is copied out.  Small problems use one panel.
    const double traffic = (double)b_bytes + (double)m * n * es_c * (beta != 0.0f ? 2.0 : 1.0);
    int64_t panel = n;
    const double wire_rate = 50e9, flop_rate = input_dtype(dtype) == GEMM_F32 ? 5.4e13 : 1.2e15;
    const double t_wire = ((double)a_bytes + (double)b_bytes + (beta != 0.0f ? (double)m * n * es_c : 0.0)) / wire_rate;
    const double t_flops = 2.0 * (double)m * (double)n * (double)k / flop_rate;
    if (traffic > 32e6 && n >= 1024) panel = host_panel_columns(input_dtype(dtype), m, n, st->sms, t_wire > 1.25 * t_flops);
    if (panel > n) panel = n;
    // While A itself is still arriving, the leading column panels are computed k panel by k panel (the order of the
    // paper's loop L2 around the packing of A, Fig. 1: C accumulates over blocks of k): each step needs only the part
    // of A that has arrived, runs on whole tiles of C, and adds onto what the earlier steps left in C.
    int64_t kpanel = k;
    // (not for 16-bit results: every step would round C to 16 bits again)
    if (panel < n && needs_ab && (double)a_bytes > 32e6 && k >= 2048 && es_c == 4) {
        int64_t kp = (int64_t)((double)a_bytes / 32e6) + 1;
        if (kp > 8) kp = 8;
        kpanel = round_up(ceil_div(k, kp), 256);
    }
    // Panel boundaries.  With k panels in play the first column panel and the first k panel are cut in two, so that the
    // first multiplication can start after half as many bytes (at 8192^3 fp32: 36 instead of 76 MB, 0.7 instead of 1.5 ms).
    std::vector<int64_t> col_edge, k_edge;
    try {
        const int64_t tile = input_dtype(dtype) == GEMM_F32 ? 128 : 256;
        for (int64_t j = 0; j < n; j += panel) {
            col_edge.push_back(j);
            if (j == 0 && kpanel < k && panel >= 4 * tile && panel < n) col_edge.push_back(round_up(panel / 2, tile));
        }
        col_edge.push_back(n);
        const int64_t kstep = kpanel > 0 ? kpanel : 1;      // k = 0: one empty k panel
        for (int64_t q = 0; q < (k > 0 ? k : 1); q += kstep) {
            k_edge.push_back(q);
            if (q == 0 && kpanel < k && kpanel >= 1024) k_edge.push_back(round_up(kpanel / 2, 256));
        }
        k_edge.push_back(k);
    } catch (...) { return GEMM_ERR_LAUNCH; }
    const int np = (int)col_edge.size() - 1, nk = (int)k_edge.size() - 1;

    void *dA = nullptr, *dB = nullptr, *dC = nullptr;
    cudaError_t e = cudaSuccess;
    int rc = GEMM_OK;
    auto chk = [&](cudaError_t r) { if (e == cudaSuccess && r != cudaSuccess) e = r; return r == cudaSuccess; };
    const size_t nev = (size_t)(3 * np + 2 * nk + 8);
    while (pipe->events.size() < nev && e == cudaSuccess) {
        cudaEvent_t ev_new;
        if (chk(cudaEventCreateWithFlags(&ev_new, cudaEventDisableTiming))) pipe->events.push_back(ev_new);
    }
    if (e != cudaSuccess) return fail_launch(e);
    cudaEvent_t* ev = pipe->events.data();
    cudaEvent_t ev_alloc = ev[0], ev_a = ev[1], ev_done = ev[2];
    size_t ev_next = 3;

    if (a_bytes) chk(cudaMallocFromPoolAsync(&dA, a_bytes, pipe->pool, s));
    if (b_bytes) chk(cudaMallocFromPoolAsync(&dB, b_bytes, pipe->pool, s));
    chk(cudaMallocFromPoolAsync(&dC, c_bytes, pipe->pool, s));
    if (e == cudaSuccess) {
        chk(cudaEventRecord(ev_alloc, s));                       // the copy streams start after the allocations
        chk(cudaStreamWaitEvent(pipe->in, ev_alloc, 0));
        chk(cudaStreamWaitEvent(pipe->out, ev_alloc, 0));
    }
    const char* hB = static_cast<const char*>(B_host);
    char* dBp = static_cast<char*>(dB);
    // columns [first column of panel pa, first column of panel pb) of C and of op(B)
    auto col0_of = [&](int p) { return col_edge[(size_t)p]; };
    auto cols_of = [&](int pa, int pb) { return col0_of(pb) - col0_of(pa); };
    auto b_off_of = [&](int p) { const int64_t j0 = col0_of(p); return needs_ab ? (tb ? (size_t)j0 * es : (size_t)j0 * ldb * es) : (size_t)0; };
    auto c_off_of = [&](int p) { return (size_t)col0_of(p) * ldc * es_c; };
    // The multiplications wait for what the inbound stream had been given when they were enqueued: the stream is in
    // order, so its latest event covers every earlier copy.
    auto arrived = [&]() {
        cudaEvent_t now = ev[ev_next++];
        chk(cudaEventRecord(now, pipe->in));
        chk(cudaStreamWaitEvent(s, now, 0));
    };
    // panels [pa, pb) of C to the device, if C is read at all (only the m rows travel: the host's padding is never touched)
    auto send_c = [&](int pa, int pb) {
        if (beta != 0.0f)
            chk(copy_window(static_cast<char*>(dC) + c_off_of(pa), static_cast<const char*>(C_host) + c_off_of(pa), m,
                            cols_of(pa, pb), ldc, es_c, cudaMemcpyHostToDevice, pipe->in));
    };
    // rows [k0, k0 + kk) of panels [pa, pb) of op(B) to the device
    auto send_b = [&](int pa, int pb, int64_t k0, int64_t kk) {
        if (!needs_ab) return;
        const size_t off = b_off_of(pa) + (tb ? (size_t)k0 * ldb * es : (size_t)k0 * es);
        if (tb) chk(copy_window(dBp + off, hB + off, cols_of(pa, pb), kk, ldb, es, cudaMemcpyHostToDevice, pipe->in));
        else chk(copy_window(dBp + off, hB + off, kk, cols_of(pa, pb), ldb, es, cudaMemcpyHostToDevice, pipe->in));
    };
    // columns [k0, k0 + kk) of op(A) to the device
    auto send_a = [&](int64_t k0, int64_t kk) {
        const size_t off = ta ? (size_t)k0 * es : (size_t)k0 * lda * es;
        char* dAp = static_cast<char*>(dA) + off;
        const char* hAp = static_cast<const char*>(A_host) + off;
        if (ta) chk(copy_window(dAp, hAp, kk, m, lda, es, cudaMemcpyHostToDevice, pipe->in));
        else chk(copy_window(dAp, hAp, m, kk, lda, es, cudaMemcpyHostToDevice, pipe->in));
    };
    // panels [pa, pb) back to the host once the multiplications enqueued so far are done
    auto return_panels = [&](int pa, int pb) {
        cudaEvent_t done = ev[ev_next++];
        chk(cudaEventRecord(done, s));
        chk(cudaStreamWaitEvent(pipe->out, done, 0));
        chk(copy_window(static_cast<char*>(C_host) + c_off_of(pa), static_cast<char*>(dC) + c_off_of(pa), m, cols_of(pa, pb),
                        ldc, es_c, cudaMemcpyDeviceToHost, pipe->out));
    };
    // columns [k0, k0 + kk) of op(A) times the matching rows of panels [pa, pb) of op(B), onto those panels of C (as one call:
    // the panels are neighbours); the first range of k applies beta, the later ones add
    auto multiply = [&](int pa, int pb, int64_t k0, int64_t kk) {
        if (e != cudaSuccess || rc != GEMM_OK) return;
        const size_t a_off = ta ? (size_t)k0 * es : (size_t)k0 * lda * es;
        const size_t bk_off = tb ? (size_t)k0 * ldb * es : (size_t)k0 * es;
        rc = gemm(dtype, transA, transB, m, cols_of(pa, pb), kk, alpha, needs_ab ? static_cast<char*>(dA) + a_off : nullptr, lda,
                  needs_ab ? dBp + b_off_of(pa) + bk_off : nullptr, ldb, k0 == 0 ? beta : 1.0f,
                  static_cast<char*>(dC) + c_off_of(pa), ldc, stream);
    };

    // Phase 1, while A arrives k panel by k panel: the first `lead` column panels are multiplied k panel by k panel.  They
    // join one after the other, a new one behind every k panel of A (its C, and the rows of its B that match the k panels
    // already there, then one multiplication over that whole range of k to catch up), so that early on, when every byte
    // on the wire enables little arithmetic, the work that can run grows in both directions at once.  From then on each k
    // panel of A travels with the matching rows of B for all panels that have joined and is multiplied into them in one call.
    int lead = 0;
    if (needs_ab) {
        lead = 1;
        if (nk > 1) {
            // every lead panel also puts its own B and C on the wire, so the arithmetic of L panels has to cover A's
            // transfer plus L panels' worth of B and C; a transfer-bound problem takes a few panels for the early overlap
            const double t_a = (double)a_bytes / wire_rate;
            const double t_panel = 2.0 * (double)m * (double)panel * (double)k / flop_rate;
            const double t_bc = ((double)panel * (double)k * es + (beta != 0.0f ? (double)m * (double)panel * es_c : 0.0)) / wire_rate;
            lead = t_panel > 1.25 * t_bc ? (int)(t_a / (t_panel - t_bc) + 0.999) : 4;
            if (col_edge[1] < panel) ++lead;          // the first panel came in two halves
            if (lead > np - 1) lead = np - 1;
            if (lead > nk) lead = nk;
            if (lead < 1) lead = 1;
        }
        send_c(0, 1);
        if (nk == 1) send_b(0, 1, 0, k);
        int joined = 1;
        for (int q = 0; q < nk && e == cudaSuccess && rc == GEMM_OK; ++q) {
            const int64_t k0 = k_edge[(size_t)q], kk = k_edge[(size_t)q + 1] - k0;
            const bool last = q == nk - 1;
            send_a(k0, kk);
            if (nk > 1) send_b(0, joined, k0, kk);
            arrived();
            if (!last) multiply(0, joined, k0, kk);
            else
                for (int p = 0; p < joined; ++p) {      // panel by panel, so that each starts home as soon as it is complete
                    multiply(p, p + 1, k0, kk);
                    return_panels(p, p + 1);
                }
            if (joined < lead) {
                send_c(joined, joined + 1);
                send_b(joined, joined + 1, 0, k0 + kk);
                arrived();
                multiply(joined, joined + 1, 0, k0 + kk);
                if (last) return_panels(joined, joined + 1);
                ++joined;
            }
        }
        lead = joined;
    }
    // Phase 2: A is resident; the remaining panels flow through copy in / multiply / copy out
    for (int p = lead; p < np && e == cudaSuccess && rc == GEMM_OK; ++p) {
        send_c(p, p + 1);
        send_b(p, p + 1, 0, k);
        arrived();
        multiply(p, p + 1, 0, k);
        if (rc != GEMM_OK) break;
        return_panels(p, p + 1);
    }
    cudaEventRecord(ev_done, pipe->out);                     // the caller's stream rejoins both copy streams
    cudaStreamWaitEvent(s, ev_done, 0);
    cudaEventRecord(ev_a, pipe->in);
    cudaStreamWaitEvent(s, ev_a, 0);
    if (dA) cudaFreeAsync(dA, s);
    if (dB) cudaFreeAsync(dB, s);
    if (dC) cudaFreeAsync(dC, s);
    chk(cudaStreamSynchronize(s));
    if (e != cudaSuccess) return fail_launch(e);
    return rc;
}

size_t gemm_workspace_bytes(int dtype, char transA, char transB, int64_t m, int64_t n, int64_t k) {
    bool ta = false, tb = false;
    const int64_t big = (int64_t)1 << 40;
    if (validate(dtype, transA, transB, m, n, k, 1.0f, (const void*)16, big, (const void*)16, big, (const void*)16, big, &ta, &tb))
        return 0;
    if (m == 0 || n == 0 || k == 0) return 0;
    DeviceState* st = device_state();
    const int sms = st ? st->sms : 148;
    // judged for 16-byte aligned pointers and minimal leading dimensions (lda = rows of the stored A, ...)
    GemmArgs a{input_dtype(dtype), ta, tb, m, n, k, 1.0f, 0.0f, (const void*)16, (const void*)16, nullptr,
               ta ? k : m, tb ? n : k, m, nullptr, nullptr};
    if (dtype == GEMM_F32_TC && split3_worthwhile(a)) {      // the pieces, then what the bfloat16 products would like
        const Split3Layout L = split3_layout(a);
        GemmArgs b = a;
        b.dtype = GEMM_BF16;
        b.lda = L.lda_p; b.ldb = L.ldb_p;
        Plan pb = make_plan(b, sms, ~(size_t)0);
        const size_t separate = L.total + (pb.kernel < 0 ? 0 : pb.ws_total);      // six launches
        return separate > L.total_fused ? separate : L.total_fused;                // one launch (pieces side by side along k)
    }
    Plan p = make_plan(a, sms, ~(size_t)0);
    return p.kernel < 0 ? 0 : p.ws_total;
}

int gemm_set_workspace(void* dev, size_t bytes, void* stream) {
    DeviceState* st = device_state();
    if (!st) return GEMM_ERR_LAUNCH;
    if (dev != nullptr && (reinterpret_cast<uintptr_t>(dev) & 255) != 0) return -1;
    cudaStream_t key = static_cast<cudaStream_t>(stream);
    Workspace w{key, dev, bytes};
    std::lock_guard<std::mutex> lock(g_mutex);
    for (size_t i = 0; i < st->ws.size(); ++i)
        if (st->ws[i].stream == key) {
            if (dev) st->ws[i] = w;
            else st->ws.erase(st->ws.begin() + (std::ptrdiff_t)i);
            return GEMM_OK;
        }
    if (dev) {
        try { st->ws.push_back(w); } catch (...) { return GEMM_ERR_LAUNCH; }
    }
    return GEMM_OK;
}

int gemm_last_config(gemm_config_t* out) {
    if (!out) return -1;
    *out = t_last_cfg;
    return GEMM_OK;
}

int gemm_force_kernel(int kernel) {
    if (kernel != GEMM_KERNEL_AUTO && kernel != GEMM_KERNEL_SIMT_GENERIC && kernel != GEMM_KERNEL_SIMT_FAST &&
        kernel != GEMM_KERNEL_TENSOR && kernel != GEMM_KERNEL_SIMT_DIRECT)
        return -1;
    g_force_kernel = kernel;
    return GEMM_OK;
}

int gemm_force_tile(int tile_m, int tile_n, int split_k) {
    if (tile_m < 0 || tile_n < 0 || split_k < 0) return -1;
    g_force_tile_m = tile_m;
    g_force_tile_n = tile_n;
    g_force_split = split_k;
    g_no_tail_split = (split_k == 1);
    return GEMM_OK;
}

int gemm_force_reduction(int how) {
    if (how < 0 || how > 2) return -1;
    g_force_reduction = how;
    return GEMM_OK;
}

int gemm_poll_status(void) {
    DeviceState* st = device_state();
    if (!st) return GEMM_ERR_LAUNCH;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return fail_launch(e);
    uint32_t word = 0;
    e = cudaMemcpy(&word, st->status, sizeof(word), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail_launch(e);
    g_last_detail.store(word);
    if (word != 0) {
        uint32_t zero = 0;
        cudaMemcpy(st->status, &zero, sizeof(zero), cudaMemcpyHostToDevice);
        return GEMM_ERR_DEVICE;
    }
    return GEMM_OK;
}

uint32_t gemm_status_detail(void) { return g_last_detail.load(); }

int gemm_selftest_wait_expiry(void* stream) {
    DeviceState* st = device_state();
    if (!st) return GEMM_ERR_LAUNCH;
    if (!st->arch_ok) return GEMM_ERR_ARCH;
    cudaError_t e = launch_wait_expiry_probe(st->status, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GEMM_OK : fail_launch(e);
}

int gemm_last_cuda_error(void) { return t_last_cuda_error; }

const char* gemm_status_string(int code) {
    switch (code) {
        case GEMM_OK: return "success";
        case GEMM_ERR_WORKSPACE: return "forced configuration needs more workspace than is registered";
        case GEMM_ERR_LAUNCH: return "CUDA runtime error (see gemm_last_cuda_error)";
        case GEMM_ERR_ARCH: return "device is not compute capability 10.x";
        case GEMM_ERR_DEVICE: return "a bounded device-side wait expired";
        case GEMM_ERR_TOO_LARGE: return "size exceeds what this entry point supports";
        case -1: return "invalid argument 1 (dtype)";
        case -2: return "invalid argument 2 (transA)";
        case -3: return "invalid argument 3 (transB)";
        case -4: return "invalid argument 4 (m)";
        case -5: return "invalid argument 5 (n)";
        case -6: return "invalid argument 6 (k)";
        case -8: return "invalid argument 8 (A)";
        case -9: return "invalid argument 9 (lda)";
        case -10: return "invalid argument 10 (B)";
        case -11: return "invalid argument 11 (ldb)";
        case -13: return "invalid argument 13 (C)";
        case -14: return "invalid argument 14 (ldc)";
        case -15: return "invalid argument 15";
        default: return "unknown status";
    }
}

}  // extern "C"
