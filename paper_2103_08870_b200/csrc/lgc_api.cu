// C ABI of liblgc: configuration checks, the carve-up of the caller's buffers, the per-step
// state machine, and the stage entry points (see include/lgc.h for the contract of each).
#include <math.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "lgc_internal.cuh"

struct lgc_ctx : lgc::Ctx {};

namespace lgc {

// Message of the calling thread's last failure that had no context to be stored in.
thread_local std::string g_last_error;
thread_local uint64_t g_kernel_launches = 0;

namespace {

constexpr size_t kAlign = 256;

// Bump allocator over the caller's scratch; with base == nullptr it only measures.
struct Carver {
    char *base;
    size_t used = 0;
    explicit Carver(void *b) : base(static_cast<char *>(b)) {}
    template <typename T>
    T *take(size_t count)
    {
        used = (used + kAlign - 1) / kAlign * kAlign;
        T *p = base ? reinterpret_cast<T *>(base + used) : nullptr;
        used += count * sizeof(T);
        return p;
    }
};

// Layers are treated per mode (Section VI-A).  Kept entries live in SLOTS: a row of `idx` holds the
// slots of the layers that go through the autoencoder first (layer order), then those of the top-k-only
// layers (layer order), so that the autoencoder's input is one contiguous vector of mu values.
// "Slot order" below means this order of the selecting layers.
struct Plan {
    int K, L, S;
    int L_ae, L_sel;                       // layers through the autoencoder / layers that select at all
    int64_t N, mu, mu_t, mu_all, muI, L1, L2, P, Penc, Pdec, code_len;   // mu: autoencoder layers' slots, mu_t: top-k-only
    int op1, op2;
    bool mixed;                            // some layer is not LGC_LAYER_TOPK_AE
    std::vector<uint8_t> mode;             // [L]
    std::vector<int> slot_layers;          // [L_sel] layers in slot order
    std::vector<int64_t> numel, off;       // [L], [L + 1]
    std::vector<int64_t> k_l, kslot;       // [L] kept entries (0: dense) and first slot (-1: dense) of every layer
    std::vector<int64_t> koff;             // [L_sel + 1] first slot of each selecting layer, slot order
    std::vector<int64_t> ki_l, kioff;      // [L_ae], [L_ae + 1] innovation counts / slots of the autoencoder layers
    std::vector<int64_t> dense_rng;        // (begin, end) of every maximal run of dense elements, ascending
};

int64_t pad4(int64_t n) { return (n + 3) / 4 * 4; }   // keeps consecutive fp32 vectors 16-byte aligned

int64_t conv_len(int64_t lin) { return lin >= 3 ? (lin - 3) / 2 + 1 : 0; }

bool ae_channels_supported(int c1, int c2)
{
    return (c1 == 8 && c2 == 4) || (c1 == 16 && c2 == 8) || (c1 == 4 && c2 == 2) || (c1 == 3 && c2 == 2);
}

lgc_status make_plan(const lgc_config *cfg, Plan &p, std::string *why)
{
    auto fail = [&](lgc_status s, const char *msg) { if (why) *why = msg; return s; };
    if (!cfg) return fail(LGC_ERR_INVALID_ARG, "config is NULL");
    if (cfg->num_nodes < 1 || cfg->num_nodes > 65535) return fail(LGC_ERR_INVALID_ARG, "num_nodes must be in [1, 65535]");
    if (cfg->num_layers < 1 || !cfg->layer_numel) return fail(LGC_ERR_INVALID_ARG, "num_layers < 1 or layer_numel is NULL");
    if (cfg->density_ppm < 1 || cfg->density_ppm > 1000000) return fail(LGC_ERR_INVALID_ARG, "density_ppm must be in [1, 10^6]");
    if (cfg->variant != LGC_VARIANT_RAR && cfg->variant != LGC_VARIANT_PS) return fail(LGC_ERR_INVALID_ARG, "unknown variant");
    if (cfg->ae_kind != LGC_AE_CONV2 && cfg->ae_kind != LGC_AE_IDENTITY && cfg->ae_kind != LGC_AE_CONV5)
        return fail(LGC_ERR_INVALID_ARG, "unknown ae_kind");
    if (!(cfg->momentum >= 0.0f && cfg->momentum < 1.0f)) return fail(LGC_ERR_INVALID_ARG, "momentum must be in [0, 1)");
    if (cfg->variant == LGC_VARIANT_PS && cfg->innovation_permille > 1000) return fail(LGC_ERR_INVALID_ARG, "innovation_permille > 1000");
    if (cfg->grad_row_stride < 0) return fail(LGC_ERR_INVALID_ARG, "grad_row_stride must not be negative");
    p.K = cfg->num_nodes;
    p.L = cfg->num_layers;
    p.S = cfg->variant == LGC_VARIANT_PS ? p.K : 1;
    p.numel.assign(cfg->layer_numel, cfg->layer_numel + p.L);
    p.mode.assign((size_t)p.L, (uint8_t)LGC_LAYER_TOPK_AE);
    p.mixed = false;
    if (cfg->layer_mode)
        for (int l = 0; l < p.L; ++l) {
            if (cfg->layer_mode[l] > LGC_LAYER_DENSE) return fail(LGC_ERR_INVALID_ARG, "unknown layer_mode");
            p.mode[l] = cfg->layer_mode[l];
            p.mixed = p.mixed || p.mode[l] != LGC_LAYER_TOPK_AE;
        }
    p.off.assign(p.L + 1, 0);
    p.k_l.assign(p.L, 0);
    p.kslot.assign(p.L, -1);
    p.dense_rng.clear();
    for (int l = 0; l < p.L; ++l) {
        const int64_t n = p.numel[l];
        if (n < 1) return fail(LGC_ERR_INVALID_ARG, "a layer has fewer than 1 element");
        p.off[l + 1] = p.off[l] + n;
        if (p.off[l + 1] > 2147483647LL) return fail(LGC_ERR_INVALID_ARG, "N exceeds 2^31 - 1");
        if (p.mode[l] == LGC_LAYER_DENSE) {
            if (!p.dense_rng.empty() && p.dense_rng.back() == p.off[l]) p.dense_rng.back() = p.off[l + 1];
            else { p.dense_rng.push_back(p.off[l]); p.dense_rng.push_back(p.off[l + 1]); }
            continue;
        }
        int64_t k = (n * (int64_t)cfg->density_ppm + 500000) / 1000000;
        p.k_l[l] = k < 1 ? 1 : (k > n ? n : k);
    }
    // slot order: the autoencoder's layers, then the top-k-only ones
    p.slot_layers.clear();
    for (int l = 0; l < p.L; ++l) if (p.mode[l] == LGC_LAYER_TOPK_AE) p.slot_layers.push_back(l);
    p.L_ae = (int)p.slot_layers.size();
    for (int l = 0; l < p.L; ++l) if (p.mode[l] == LGC_LAYER_TOPK_ONLY) p.slot_layers.push_back(l);
    p.L_sel = (int)p.slot_layers.size();
    if (p.L_ae == 0)
        return fail(LGC_ERR_INVALID_ARG, "no layer has LGC_LAYER_TOPK_AE: at least one layer must feed the autoencoder");
    p.koff.assign(p.L_sel + 1, 0);
    p.ki_l.assign(p.L_ae, 0);
    p.kioff.assign(p.L_ae + 1, 0);
    for (int j = 0; j < p.L_sel; ++j) {
        const int l = p.slot_layers[j];
        p.kslot[l] = p.koff[j];
        p.koff[j + 1] = p.koff[j] + p.k_l[l];
        if (j < p.L_ae) {
            int64_t ki = (p.k_l[l] * (int64_t)cfg->innovation_permille + 500) / 1000;
            ki = ki < 1 ? 1 : (ki > p.k_l[l] ? p.k_l[l] : ki);
            p.ki_l[j] = ki;
            p.kioff[j + 1] = p.kioff[j] + ki;
        }
    }
    p.N = p.off[p.L];
    if (cfg->grad_row_stride != 0 && cfg->grad_row_stride < p.N) return fail(LGC_ERR_INVALID_ARG, "grad_row_stride is smaller than N");
    p.mu = p.koff[p.L_ae];
    p.mu_all = p.koff[p.L_sel];
    p.mu_t = p.mu_all - p.mu;
    p.muI = p.kioff[p.L_ae];
    p.L1 = conv_len(p.mu);
    p.L2 = conv_len(p.L1);
    p.op1 = p.L1 >= 3 ? (int)((p.L1 - 3) % 2) : 0;
    p.op2 = p.mu >= 3 ? (int)((p.mu - 3) % 2) : 0;
    if (cfg->ae_kind == LGC_AE_CONV2) {
        if (!ae_channels_supported(cfg->ae_c1, cfg->ae_c2))
            return fail(LGC_ERR_UNSUPPORTED, "autoencoder channels must be (8,4), (16,8), (4,2) or (3,2)");
        if (p.L2 < 1) return fail(LGC_ERR_UNSUPPORTED, "mu is too short for two stride-2 convolutions (needs mu >= 7)");
        const int64_t c1 = cfg->ae_c1, c2 = cfg->ae_c2;
        p.Penc = c1 * 3 + c1 + c2 * c1 * 3 + c2;
        p.Pdec = c2 * c1 * 3 + c1 + c1 * 3 + 1 + (cfg->variant == LGC_VARIANT_PS ? 3 : 0);
        p.P = p.Penc + p.Pdec * p.S;
        p.code_len = c2 * p.L2;
    } else if (cfg->ae_kind == LGC_AE_CONV5) {
        int64_t len[5];
        if (!ae5_lengths(p.mu, len) || len[4] < 1) return fail(LGC_ERR_UNSUPPORTED, "mu is too short for four stride-2 convolutions (needs mu >= 31)");
        p.P = ae5_param_count(p.S, cfg->variant == LGC_VARIANT_PS);
        p.Penc = p.Pdec = 0;
        p.code_len = 4 * len[4];
    } else {
        p.Penc = p.Pdec = p.P = 0;
        p.code_len = p.mu;
    }
    return LGC_OK;
}

// Host-side description of one selection family: which segments are small or large, and how the
// large ones are cut by the row's tiles of kSelChunk elements.
struct SelectPlan {
    std::vector<int64_t> seg_off, comp_off;
    std::vector<int32_t> seg_len, seg_k, seg_out, small_ids, large_ids, seg_large, large_q0, large_order, tchunk0,
        tchunk_large;
    std::vector<int4> tile_desc;
    std::vector<int2> group_job;
    int tiles_per_row = 0;
    int64_t comp_total = 0;
};

// Segments ascend by offset and may leave gaps (layers that do not select).  row_len: length of a row;
// dense: (begin, end) pairs of the row's dense runs, ascending (they lie in the gaps).
SelectPlan plan_select(const std::vector<int64_t> &off, const std::vector<int64_t> &len, const std::vector<int64_t> &k,
                       const std::vector<int64_t> &out_off, int64_t row_len, const std::vector<int64_t> &dense)
{
    SelectPlan sp;
    const int n = (int)len.size();
    sp.comp_off.push_back(0);
    sp.tchunk0.push_back(0);
    for (int i = 0; i < n; ++i) {
        sp.seg_off.push_back(off[i]);
        sp.seg_len.push_back((int32_t)len[i]);
        sp.seg_k.push_back((int32_t)k[i]);
        sp.seg_out.push_back((int32_t)out_off[i]);
        if (len[i] <= kSelChunk) {
            sp.small_ids.push_back(i);
            sp.seg_large.push_back(-1);
        } else {
            const int li = (int)sp.large_ids.size();
            sp.large_ids.push_back(i);
            sp.seg_large.push_back(li);
            const int64_t q0 = off[i] / kSelChunk, q1 = (off[i] + len[i] - 1) / kSelChunk;
            sp.large_q0.push_back((int32_t)q0);
            for (int64_t q = q0; q <= q1; ++q) sp.tchunk_large.push_back(li);
            const int32_t c0 = sp.tchunk0.back(), c1 = (int32_t)sp.tchunk_large.size();
            if (c1 - c0 > kSelGroup)
                for (int32_t gb = c0; gb < c1; gb += kSelGroup) sp.group_job.push_back(make_int2(li, gb));
            sp.tchunk0.push_back(c1);
            sp.comp_off.push_back(sp.comp_off.back() + select_compact_capacity(len[i], k[i]));
        }
    }
    sp.comp_total = sp.comp_off.back();
    sp.large_order.resize(sp.large_ids.size());
    for (size_t i = 0; i < sp.large_order.size(); ++i) sp.large_order[i] = (int32_t)i;
    std::stable_sort(sp.large_order.begin(), sp.large_order.end(), [&](int32_t a, int32_t b) {
        return len[sp.large_ids[a]] > len[sp.large_ids[b]];
    });
    sp.tiles_per_row = (int)((row_len + kSelChunk - 1) / kSelChunk);
    int s = 0;
    size_t d0 = 0;                                                  // first dense run that ends after the tile's start
    for (int q = 0; q < sp.tiles_per_row; ++q) {
        const int64_t t0 = (int64_t)q * kSelChunk, t1 = t0 + kSelChunk < row_len ? t0 + kSelChunk : row_len;
        while (s < n && off[s] + len[s] <= t0) ++s;                 // first segment that reaches into tile q or lies behind it
        int4 d = make_int4(s, -2, 0, 0);
        if (s < n && off[s] <= t0 && off[s] + len[s] >= t1 && sp.seg_large[s] >= 0) {
            d.y = sp.seg_large[s];                                  // one large segment covers the tile
            d.z = sp.tchunk0[d.y] + (q - sp.large_q0[d.y]);
        } else {
            for (int r = s; r < n && off[r] < t1; ++r)
                if (sp.seg_large[r] >= 0) d.y = -1;                 // several segments, at least one large
        }
        while (d0 < dense.size() && dense[d0 + 1] <= t0) d0 += 2;
        if (d0 < dense.size() && dense[d0] < t1) {
            // w: 0 no dense element in the tile; one dense run [lo, hi) (positions inside the tile): 1 + lo + (hi << 13);
            // several runs: -(1 + the first one's number)
            if (d0 + 2 < dense.size() && dense[d0 + 2] < t1) {
                d.w = -((int)(d0 / 2) + 1);
            } else {
                const int lo = (int)(std::max<int64_t>(dense[d0], t0) - t0), hi = (int)(std::min<int64_t>(dense[d0 + 1], t1) - t0);
                d.w = 1 + lo + (hi << 13);
            }
        }
        sp.tile_desc.push_back(d);
    }
    return sp;
}

// The two selection families of a context: the residual v over the selecting layers (layer order; slots
// as the plan assigns them), and -- parameter server -- the kept values of the autoencoder layers.
SelectPlan plan_select_v(const Plan &p)
{
    std::vector<int64_t> off, len, k, out;
    for (int l = 0; l < p.L; ++l)
        if (p.mode[l] != LGC_LAYER_DENSE) {
            off.push_back(p.off[l]); len.push_back(p.numel[l]); k.push_back(p.k_l[l]); out.push_back(p.kslot[l]);
        }
    return plan_select(off, len, k, out, p.N, p.dense_rng);
}
SelectPlan plan_select_inn(const Plan &p)
{
    std::vector<int64_t> off(p.koff.begin(), p.koff.begin() + p.L_ae), len, out(p.kioff.begin(), p.kioff.begin() + p.L_ae);
    for (int j = 0; j < p.L_ae; ++j) len.push_back(p.k_l[p.slot_layers[j]]);
    return plan_select(off, len, p.ki_l, out, p.mu, {});
}

void carve_select(Carver &cv, SelectTables &t, const SelectPlan &sp, int rows)
{
    const int S = (int)sp.seg_len.size(), ns = (int)sp.small_ids.size(), nl = (int)sp.large_ids.size();
    const int nc = (int)sp.tchunk_large.size();
    t.num_segments = S; t.num_small = ns; t.num_large = nl; t.num_tchunks = nc; t.tiles_per_row = sp.tiles_per_row;
    t.max_rows = rows;
    t.seg_off = cv.take<int64_t>(S);
    t.seg_len = cv.take<int32_t>(S);
    t.seg_k = cv.take<int32_t>(S);
    t.seg_out = cv.take<int32_t>(S);
    t.seg_large = cv.take<int32_t>(S);
    t.small_ids = cv.take<int32_t>(ns);
    t.large_ids = cv.take<int32_t>(nl);
    t.large_q0 = cv.take<int32_t>(nl);
    t.large_order = cv.take<int32_t>(nl);
    t.tchunk0 = cv.take<int32_t>(nl + 1);
    t.tchunk_large = cv.take<int32_t>(nc);
    t.tile_desc = cv.take<int4>(sp.tiles_per_row);
    t.num_group_jobs = (int)sp.group_job.size();
    t.group_job = cv.take<int2>(sp.group_job.size());
    t.job_range = cv.take<int2>((size_t)rows * sp.group_job.size());
    t.job_cnt = cv.take<int2>((size_t)rows * sp.group_job.size());
    t.seg_wide = cv.take<int32_t>((size_t)rows * nl);
    t.hist = cv.take<uint32_t>((size_t)rows * nl * kHistBins);
    t.prefix = cv.take<uint32_t>((size_t)rows * nl);
    t.k_rem = cv.take<int32_t>((size_t)rows * nl);
    t.seg_m = cv.take<int32_t>((size_t)rows * nl);
    t.seg_ticket = cv.take<int32_t>((size_t)rows * nl);
    t.seg_epoch = cv.take<int32_t>((size_t)rows * nl);
    t.lbkey = cv.take<uint32_t>((size_t)rows * nl);
    t.last_key = cv.take<uint32_t>((size_t)rows * nl);
    t.key_trend = cv.take<float2>((size_t)rows * nl);
    t.seg_path = cv.take<int32_t>((size_t)rows * nl);
    t.cand_cnt = cv.take<int32_t>((size_t)rows * nc);
    t.cand = cv.take<uint2>((size_t)rows * nc * kSelCandCap);
    t.comp_off = cv.take<int64_t>((size_t)nl + 1);
    t.comp_total = sp.comp_total;
    t.comp_key = cv.take<uint32_t>((size_t)rows * sp.comp_total);
    t.comp_idx = cv.take<int32_t>((size_t)rows * sp.comp_total);
}

// Lays every sub-buffer of the scratch out; identical for measuring and for real.
void carve(Carver &cv, Ctx &c, const Plan &p, const lgc_config &cfg)
{
    const bool ps = cfg.variant == LGC_VARIANT_PS;
    const bool conv = cfg.ae_kind == LGC_AE_CONV2;
    const bool conv5 = cfg.ae_kind == LGC_AE_CONV5;
    c.errword = cv.take<int32_t>(4);
    c.idx = cv.take<int32_t>((size_t)p.S * p.mu_all);
    c.val = cv.take<float>((size_t)p.K * p.mu);
    c.val_t = p.mu_t ? cv.take<float>((size_t)p.K * p.mu_t) : nullptr;
    c.num_dense = (int)(p.dense_rng.size() / 2);
    c.num_dense_chunks = 0;
    for (size_t r = 0; r < p.dense_rng.size(); r += 2)
        c.num_dense_chunks += (p.dense_rng[r + 1] - p.dense_rng[r] + kDenseChunk - 1) / kDenseChunk;
    c.dense_rng = c.num_dense ? cv.take<int64_t>(p.dense_rng.size()) : nullptr;
    c.dense_chunks = c.num_dense ? cv.take<int64_t>((size_t)2 * c.num_dense_chunks) : nullptr;
    c.code = conv || conv5 ? cv.take<float>((size_t)p.K * p.code_len) : nullptr;
    c.combined = cv.take<float>((size_t)p.code_len);
    c.recon = cv.take<float>((size_t)p.S * p.mu);
    c.slot_layer = cv.take<int32_t>((size_t)p.mu_all);
    c.koff_dev = cv.take<int32_t>((size_t)p.L + 1);
    c.layer_off_dev = cv.take<int64_t>((size_t)p.L);
    c.ic_bytes = cv.take<unsigned char>((size_t)5 * p.mu_all);
    c.tile_lo = cv.take<int32_t>((size_t)((p.N + 4095) / 4096) + 1);
    carve_select(cv, c.sel_v, plan_select_v(p), p.S);
    c.sel_v.dense_rng = c.dense_rng;
    c.sel_v.num_dense = c.num_dense;
    if (ps) {
        c.inn = cv.take<float>((size_t)p.K * p.mu);
        c.inn_pos = cv.take<int32_t>((size_t)p.K * p.muI);
        c.inn_slot_layer = cv.take<int32_t>((size_t)p.muI);
        c.kioff_dev = cv.take<int32_t>((size_t)p.L + 1);
        c.koff64_dev = cv.take<int64_t>((size_t)p.L);
        carve_select(cv, c.sel_inn, plan_select_inn(p), p.K);
    }
    if (conv && ps) {                       // training work space, one slice per node
        const size_t c1 = cfg.ae_c1, c2 = cfg.ae_c2, K = p.K;
        c.t_h = cv.take<float>(K * c1 * p.L1);
        c.t_dh = cv.take<float>(K * c1 * p.L1);
        c.t_d = cv.take<float>(K * c1 * p.L1);
        c.t_dd = cv.take<float>(K * c1 * p.L1);
        c.t_dr = cv.take<float>(K * p.mu);
        c.t_y = cv.take<float>(K * p.mu);
        c.t_dy = cv.take<float>(K * p.mu);
        c.t_dz = cv.take<float>(K * c2 * p.L2);
        c.t_dzc = cv.take<float>(K * c2 * p.L2);
        c.t_zsum = cv.take<float>(c2 * p.L2);
        c.t_loss_blocks = (int)((p.mu + 127) / 128);
        c.t_loss_part = cv.take<double>(K * (size_t)c.t_loss_blocks);
        c.t_sim_part = cv.take<double>((size_t)((p.L2 + 127) / 128));
    }
    if (conv && !ps) {
        const size_t c1 = cfg.ae_c1, c2 = cfg.ae_c2;
        c.t_h = cv.take<float>((size_t)p.K * c1 * p.L1);
        c.t_dh = cv.take<float>((size_t)p.K * c1 * p.L1);
        c.t_d = cv.take<float>(c1 * p.L1);
        c.t_dd = cv.take<float>(c1 * p.L1);
        c.t_dr = cv.take<float>((size_t)p.mu);
        c.t_dz = cv.take<float>(c2 * p.L2);
        c.t_loss_blocks = (int)((p.mu + 127) / 128);
        c.t_loss_part = cv.take<double>((size_t)c.t_loss_blocks);
    }
    if (conv5) {
        if (!c.ae5) c.ae5.reset(new Ae5());
        ae5_carve(*c.ae5, p.K, p.mu, ps, cv.base, &cv.used);
    }
    cv.take<char>(0);
}

lgc_status fail(lgc_ctx *ctx, lgc_status s, const std::string &msg)
{
    if (ctx) ctx->err = msg;
    else g_last_error = msg;
    return s;
}

lgc_status cuda_fail(lgc_ctx *ctx, cudaError_t e, const char *where)
{
    return fail(ctx, LGC_ERR_CUDA, std::string(where) + ": " + cudaGetErrorString(e));
}

template <typename T>
cudaError_t upload(T *dst, const std::vector<T> &src, cudaStream_t s)
{
    if (src.empty()) return cudaSuccess;
    return cudaMemcpyAsync(dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice, s);
}

// Uploads the tables of one selection family; `hold` keeps the host copies alive until the
// stream has been synchronised.
cudaError_t upload_select(SelectTables &t, SelectPlan sp, cudaStream_t s, std::vector<SelectPlan> &hold)
{
    hold.push_back(std::move(sp));
    const SelectPlan &h = hold.back();
    cudaError_t e = upload(t.seg_off, h.seg_off, s);
    if (e == cudaSuccess) e = upload(t.comp_off, h.comp_off, s);
    if (e == cudaSuccess) e = upload(t.tile_desc, h.tile_desc, s);
    if (e == cudaSuccess) e = upload(t.group_job, h.group_job, s);
    const std::vector<int32_t> *arrs[] = {&h.seg_len, &h.seg_k, &h.seg_out, &h.seg_large, &h.small_ids, &h.large_ids,
                                          &h.large_q0, &h.large_order, &h.tchunk0, &h.tchunk_large};
    int32_t *dsts[] = {t.seg_len, t.seg_k, t.seg_out, t.seg_large, t.small_ids, t.large_ids,
                       t.large_q0, t.large_order, t.tchunk0, t.tchunk_large};
    for (int i = 0; i < 10 && e == cudaSuccess; ++i) e = upload(dsts[i], *arrs[i], s);
    return e;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace
}  // namespace lgc

using namespace lgc;

extern "C" {

lgc_status lgc_workspace_bytes(const lgc_config *cfg, size_t *state_bytes, size_t *scratch_bytes, size_t *params_bytes)
{
    Plan p;
    const lgc_status st = make_plan(cfg, p, nullptr);
    if (st != LGC_OK) return st;
    Ctx tmp;
    Carver cv(nullptr);
    carve(cv, tmp, p, *cfg);
    if (state_bytes) *state_bytes = (size_t)2 * pad4((int64_t)p.K * p.N) * sizeof(float);
    if (scratch_bytes) *scratch_bytes = (cv.used + kAlign - 1) / kAlign * kAlign;
    if (params_bytes) *params_bytes = (size_t)(p.P > 0 ? 3 * pad4(p.P) : 4) * sizeof(float);
    return LGC_OK;
}

lgc_status lgc_init(const lgc_config *cfg, void *state, size_t state_bytes, void *scratch, size_t scratch_bytes,
                    void *params, size_t params_bytes, lgc_ctx **out)
{
    if (!out) return LGC_ERR_INVALID_ARG;
    *out = nullptr;
    Plan p;
    lgc_status st = make_plan(cfg, p, nullptr);
    if (st != LGC_OK) return st;
    size_t need_state, need_scratch, need_params;
    lgc_workspace_bytes(cfg, &need_state, &need_scratch, &need_params);
    if (!state || !scratch || !params || !aligned16(state) || !aligned16(scratch) || !aligned16(params))
        return LGC_ERR_INVALID_ARG;
    if (state_bytes < need_state || scratch_bytes < need_scratch || params_bytes < need_params) return LGC_ERR_WORKSPACE;

    lgc_ctx *c = new (std::nothrow) lgc_ctx();
    if (!c) return LGC_ERR_NO_MEMORY;
    c->cfg = *cfg;
    c->cfg.layer_numel = nullptr;
    c->cfg.layer_mode = nullptr;
    c->stream = static_cast<cudaStream_t>(cfg->stream);
    c->K = p.K; c->L = p.L; c->S = p.S; c->N = p.N; c->mu = p.mu; c->muI = p.muI; c->L1 = p.L1; c->L2 = p.L2;
    c->mu_t = p.mu_t; c->mu_all = p.mu_all; c->mixed = p.mixed; c->L_ae = p.L_ae; c->L_sel = p.L_sel;
    c->P = p.P; c->Penc = p.Penc; c->Pdec = p.Pdec; c->op1 = p.op1; c->op2 = p.op2; c->code_len = p.code_len;
    c->numel = p.numel; c->off = p.off; c->k_l = p.k_l; c->kslot = p.kslot; c->koff = p.koff; c->ki_l = p.ki_l; c->kioff = p.kioff;
    c->lr = cfg->adam_lr != 0.0f ? (double)cfg->adam_lr : 1e-3;
    c->beta1 = cfg->adam_beta1 != 0.0f ? (double)cfg->adam_beta1 : 0.9;
    c->beta2 = cfg->adam_beta2 != 0.0f ? (double)cfg->adam_beta2 : 0.999;
    c->eps = cfg->adam_eps != 0.0f ? (double)cfg->adam_eps : 1e-8;
    c->u = static_cast<float *>(state);
    c->v = c->u + pad4((int64_t)p.K * p.N);   // both halves start 16-byte aligned
    c->params = static_cast<float *>(params);
    c->adam_m = c->params + pad4(p.P);
    c->adam_v = c->adam_m + pad4(p.P);
    Carver cv(scratch);
    carve(cv, *c, p, *cfg);
    if (cfg->ae_kind == LGC_AE_IDENTITY) c->code = c->val;

    cudaStream_t s = c->stream;
    cudaError_t e = launch_zero(state, need_state, s);
    if (e == cudaSuccess) e = launch_zero(scratch, need_scratch, s);
    if (e == cudaSuccess && p.P > 0) e = launch_zero(c->adam_m, (size_t)2 * pad4(p.P) * sizeof(float), s);
    std::vector<SelectPlan> hold;
    hold.reserve(2);
    if (e == cudaSuccess) e = upload_select(c->sel_v, plan_select_v(p), s, hold);
    if (e == cudaSuccess && cfg->variant == LGC_VARIANT_PS)
        e = upload_select(c->sel_inn, plan_select_inn(p), s, hold);
    // tables in slot order (the autoencoder's layers first): layer of every slot, first slot and first element of every layer
    std::vector<int32_t> slot_layer((size_t)p.mu_all), koff32((size_t)p.L_sel + 1);
    std::vector<int64_t> layer_off((size_t)p.L_sel);
    for (int j = 0; j < p.L_sel; ++j) {
        koff32[j] = (int32_t)p.koff[j];
        layer_off[j] = p.off[p.slot_layers[j]];
        for (int64_t q = p.koff[j]; q < p.koff[j + 1]; ++q) slot_layer[(size_t)q] = j;
    }
    koff32[p.L_sel] = (int32_t)p.mu_all;
    if (e == cudaSuccess) e = upload(c->slot_layer, slot_layer, s);
    if (e == cudaSuccess) e = upload(c->koff_dev, koff32, s);
    if (e == cudaSuccess) e = upload(c->layer_off_dev, layer_off, s);
    std::vector<int64_t> dense_chunks;
    for (size_t r = 0; r < p.dense_rng.size(); r += 2)
        for (int64_t a = p.dense_rng[r]; a < p.dense_rng[r + 1]; a += kDenseChunk) {
            dense_chunks.push_back(a);
            dense_chunks.push_back(std::min<int64_t>(a + kDenseChunk, p.dense_rng[r + 1]));
        }
    if (e == cudaSuccess) e = upload(c->dense_rng, p.dense_rng, s);
    if (e == cudaSuccess) e = upload(c->dense_chunks, dense_chunks, s);
    std::vector<int32_t> inn_slot_layer, kioff32;
    std::vector<int64_t> koff64;
    if (cfg->variant == LGC_VARIANT_PS) {
        inn_slot_layer.resize((size_t)p.muI);
        kioff32.resize((size_t)p.L_ae + 1);
        koff64.assign(p.koff.begin(), p.koff.begin() + p.L_ae);
        for (int j = 0; j < p.L_ae; ++j) {
            kioff32[j] = (int32_t)p.kioff[j];
            for (int64_t q = p.kioff[j]; q < p.kioff[j + 1]; ++q) inn_slot_layer[(size_t)q] = j;
        }
        kioff32[p.L_ae] = (int32_t)p.muI;
        if (e == cudaSuccess) e = upload(c->inn_slot_layer, inn_slot_layer, s);
        if (e == cudaSuccess) e = upload(c->kioff_dev, kioff32, s);
        if (e == cudaSuccess) e = upload(c->koff64_dev, koff64, s);
    }
    if (e == cudaSuccess && cfg->ae_kind == LGC_AE_CONV5) e = ae5_make_maps(*c);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        delete c;
        cudaGetLastError();
        return cuda_fail(nullptr, e, "lgc_init");
    }
    *out = c;
    return LGC_OK;
}

lgc_status lgc_destroy(lgc_ctx *ctx)
{
    if (ctx) {
        for (cudaEvent_t e : ctx->row_uploaded) cudaEventDestroy(e);
        if (ctx->tail_done) cudaEventDestroy(ctx->tail_done);
        if (ctx->upload_stream) cudaStreamDestroy(ctx->upload_stream);
        if (ctx->side_fork) cudaEventDestroy(ctx->side_fork);
        if (ctx->side_join) cudaEventDestroy(ctx->side_join);
        if (ctx->side_stream) cudaStreamDestroy(ctx->side_stream);
    }
    delete ctx;
    return LGC_OK;
}

namespace {

// Opens a step: checks, advances the step counter and decides whether the accumulation also collects
// selection candidates.  The fused form needs rows that start 16-byte aligned, someone to select for,
// and the keys two previous selections left to collect against (one key says where the threshold was,
// two how fast it moves).
lgc_status open_step(lgc_ctx *c, const float *grads, int32_t leader_hint, bool *fused)
{
    if (!grads || !aligned16(grads)) return fail(c, LGC_ERR_INVALID_ARG, "grads is NULL or not 16-byte aligned");
    if (c->stage != Ctx::kIdle) return fail(c, LGC_ERR_BAD_STATE, "lgc_accumulate must open a step");
    const bool ps = c->cfg.variant == LGC_VARIANT_PS;
    if (!ps && leader_hint >= c->K) return fail(c, LGC_ERR_INVALID_ARG, "leader_hint out of range");
    c->epoch = c->epoch == 0x7fffffff ? 1 : c->epoch + 1;
    c->cleared_update = nullptr;
    const int64_t gs = c->cfg.grad_row_stride ? c->cfg.grad_row_stride : c->N;
    *fused = c->N % 4 == 0 && gs % 4 == 0 && c->sel_v.num_large > 0 && c->selections >= 2 && (ps || leader_hint >= 0);
    c->fused_leader = *fused ? (ps ? -1 : leader_hint) : -2;
    return LGC_OK;
}

// Stage 1 for the nodes r0 .. r1 - 1 of an opened step.  Every element is updated by the same two
// operations whichever kernel and however many launches serve it.
cudaError_t accumulate_nodes(lgc_ctx *c, const float *grads, int32_t leader_hint, bool fused, int r0, int r1)
{
    const bool ps = c->cfg.variant == LGC_VARIANT_PS;
    const int64_t gs = c->cfg.grad_row_stride ? c->cfg.grad_row_stride : c->N;
    const float *g = grads + (int64_t)r0 * gs;
    float *u = c->u + (int64_t)r0 * c->N, *v = c->v + (int64_t)r0 * c->N;
    if (fused)   // the kernel's row y is node r0 + y; node n selects into table row n (parameter server) or 0 (the leader)
        return launch_accumulate_select(c->sel_v, g, gs, u, v, r1 - r0, c->N, c->cfg.momentum, (ps ? 0 : leader_hint) - r0,
                                        ps ? c->K : 1, c->epoch, c->errword, c->stream);
    if (c->num_dense && c->N % 4 == 0 && gs % 4 == 0)      // the tile kernel, nobody selecting: it skips the dense layers
        return launch_accumulate_select(c->sel_v, g, gs, u, v, r1 - r0, c->N, c->cfg.momentum, 0, 0, c->epoch, c->errword,
                                        c->stream);
    if (gs == c->N && r0 == 0 && r1 == c->K && !c->num_dense)
        return launch_accumulate(g, u, v, (uint64_t)c->K * (uint64_t)c->N, c->cfg.momentum, c->stream);
    return launch_accumulate_rows(g, gs, u, v, r1 - r0, c->N, c->cfg.momentum, c->dense_rng, c->num_dense, c->stream);
}

}  // namespace

lgc_status lgc_accumulate(lgc_ctx *c, const float *grads, int32_t leader_hint)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    bool fused;
    const lgc_status st = open_step(c, grads, leader_hint, &fused);
    if (st != LGC_OK) return st;
    const cudaError_t e = accumulate_nodes(c, grads, leader_hint, fused, 0, c->K);
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_accumulate");
    c->step_grads = grads;
    c->tail_recorded = false;      // a later lgc_step_host orders its upload behind this step
    c->stage = Ctx::kAccumulated;
    return LGC_OK;
}

lgc_status lgc_topk(lgc_ctx *c, int32_t leader, float *update_hint)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (c->stage != Ctx::kAccumulated) return fail(c, LGC_ERR_BAD_STATE, "lgc_topk must follow lgc_accumulate");
    if (update_hint && !aligned16(update_hint)) return fail(c, LGC_ERR_INVALID_ARG, "update_hint is not 16-byte aligned");
    const bool ps = c->cfg.variant == LGC_VARIANT_PS;
    if (!ps && (leader < 0 || leader >= c->K)) return fail(c, LGC_ERR_INVALID_ARG, "leader out of range");
    // candidates collected during the accumulation count only if they are this leader's
    const bool served = ps ? c->fused_leader == -1 : c->fused_leader == leader;
    cudaError_t e = cudaSuccess;
    if (ps && !c->side_stream && c->sel_v.num_small && c->sel_v.num_large) {     // many small layers: a stream for them
        e = cudaStreamCreateWithFlags(&c->side_stream, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->side_fork, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->side_join, cudaEventDisableTiming);
        if (e != cudaSuccess) return cuda_fail(c, e, "lgc_topk (side stream)");
    }
    e = launch_select(c->sel_v, c->v, c->N, ps ? 0 : leader, c->S, c->idx, c->mu_all, served, c->epoch, update_hint, c->N,
                      c->errword, c->stream, c->side_stream, c->side_fork, c->side_join);
    c->cleared_update = c->sel_v.num_large ? update_hint : nullptr;
    if (c->selections < 2) ++c->selections;
    c->val_valid = false;
    c->mean_valid = false;
    c->tile_lo_valid = false;
    // ring-allreduce with the convolutional autoencoder gathers inside the encoder launch
    if (e == cudaSuccess && (ps || c->cfg.ae_kind == LGC_AE_IDENTITY)) e = launch_gather(*c);
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_topk");
    c->last_leader = leader;
    c->stage = Ctx::kSelected;
    return LGC_OK;
}

lgc_status lgc_encode(lgc_ctx *c)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (c->stage != Ctx::kSelected) return fail(c, LGC_ERR_BAD_STATE, "lgc_encode must follow lgc_topk");
    const cudaError_t e = launch_encode(*c);
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_encode");
    c->stage = Ctx::kEncoded;
    return LGC_OK;
}

lgc_status lgc_combine(lgc_ctx *c, int32_t common_node)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (c->stage != Ctx::kEncoded) return fail(c, LGC_ERR_BAD_STATE, "lgc_combine must follow lgc_encode");
    cudaError_t e;
    if (c->cfg.variant == LGC_VARIANT_PS) {
        if (common_node < 0 || common_node >= c->K) return fail(c, LGC_ERR_INVALID_ARG, "common_node out of range");
        e = launch_combine_ps(*c, common_node);
    } else {
        e = launch_combine_mean(*c);
    }
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_combine");
    c->stage = Ctx::kCombined;
    return LGC_OK;
}

lgc_status lgc_decode_scatter(lgc_ctx *c, float *update)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (!update || !aligned16(update)) return fail(c, LGC_ERR_INVALID_ARG, "update is NULL or not 16-byte aligned");
    if (c->stage != Ctx::kCombined) return fail(c, LGC_ERR_BAD_STATE, "lgc_decode_scatter must follow lgc_combine");
    const cudaError_t e = launch_decode_scatter(*c, update);
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_decode_scatter");
    c->stage = Ctx::kIdle;
    return LGC_OK;
}

lgc_status lgc_topk_scatter(lgc_ctx *c, float *update)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (!update || !aligned16(update)) return fail(c, LGC_ERR_INVALID_ARG, "update is NULL or not 16-byte aligned");
    if (c->stage != Ctx::kSelected) return fail(c, LGC_ERR_BAD_STATE, "lgc_topk_scatter must follow lgc_topk");
    const cudaError_t e = launch_topk_scatter(*c, update);
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_topk_scatter");
    c->stage = Ctx::kIdle;
    return LGC_OK;
}

lgc_status lgc_abort_step(lgc_ctx *c)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    c->stage = Ctx::kIdle;
    c->cleared_update = nullptr;
    c->fused_leader = -2;
    c->val_valid = c->mean_valid = c->tile_lo_valid = false;
    return LGC_OK;
}

lgc_status lgc_ae_train_step(lgc_ctx *c, float *loss_out)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (c->cfg.variant != LGC_VARIANT_RAR || c->cfg.ae_kind == LGC_AE_IDENTITY)
        return fail(c, LGC_ERR_UNSUPPORTED, "training is built for the ring-allreduce convolutional autoencoders");
    if (c->stage != Ctx::kSelected) return fail(c, LGC_ERR_BAD_STATE, "lgc_ae_train_step must follow lgc_topk");
    cudaError_t e;
    if (c->cfg.ae_kind == LGC_AE_CONV5) {
        e = launch_ae5_train_step(*c, loss_out);       // its first convolution gathers the kept values itself
    } else {
        e = launch_gather(*c);
        if (e == cudaSuccess) e = launch_train_step(*c, loss_out);
    }
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_ae_train_step");
    return LGC_OK;
}

lgc_status lgc_ae_train_step_ps(lgc_ctx *c, int32_t common_node, float lambda_rec, float lambda_sim, float *loss_out)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (c->cfg.variant != LGC_VARIANT_PS || c->cfg.ae_kind == LGC_AE_IDENTITY)
        return fail(c, LGC_ERR_UNSUPPORTED, "lgc_ae_train_step_ps needs the parameter-server variant with a convolutional autoencoder");
    if (common_node < 0 || common_node >= c->K) return fail(c, LGC_ERR_INVALID_ARG, "common_node out of range");
    if (!(lambda_rec >= 0.0f) || !(lambda_sim >= 0.0f)) return fail(c, LGC_ERR_INVALID_ARG, "the loss weights must not be negative");
    if (c->stage != Ctx::kSelected) return fail(c, LGC_ERR_BAD_STATE, "lgc_ae_train_step_ps must follow lgc_topk");
    cudaError_t e = launch_gather(*c);
    if (e == cudaSuccess)
        e = c->cfg.ae_kind == LGC_AE_CONV5 ? launch_ae5_train_step_ps(*c, common_node, lambda_rec, lambda_sim, loss_out)
                                           : launch_train_step_ps(*c, common_node, lambda_rec, lambda_sim, loss_out);
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_ae_train_step_ps");
    return LGC_OK;
}

lgc_status lgc_dense_mean(const float *grads, int64_t row_stride, int32_t num_nodes, int64_t n, float *update, void *stream)
{
    if (!grads || !update || num_nodes < 1 || n < 0 || (num_nodes > 1 && row_stride < n)) {
        g_last_error = "lgc_dense_mean: NULL buffer, no nodes, or rows that overlap";
        return LGC_ERR_INVALID_ARG;
    }
    const cudaError_t e = launch_dense_mean(grads, row_stride, num_nodes, n, update, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(nullptr, e, "lgc_dense_mean");
    return LGC_OK;
}

lgc_status lgc_encode_indices(lgc_ctx *c, int32_t node, void *stream_out, size_t capacity, uint64_t *sizes_out)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (!stream_out || !sizes_out || capacity < 4 || capacity % 4 != 0 || (reinterpret_cast<uintptr_t>(stream_out) & 3) != 0 ||
        (reinterpret_cast<uintptr_t>(sizes_out) & 7) != 0)
        return fail(c, LGC_ERR_INVALID_ARG, "lgc_encode_indices: buffers must be non-NULL, the stream 4-byte aligned with a capacity that is a multiple of 4");
    if (c->stage == Ctx::kIdle || c->stage == Ctx::kAccumulated)
        return fail(c, LGC_ERR_BAD_STATE, "lgc_encode_indices needs the index sets of this step's lgc_topk");
    if (c->cfg.variant == LGC_VARIANT_PS ? (node < 0 || node >= c->K) : node != 0 && (node < 0 || node >= c->K))
        return fail(c, LGC_ERR_INVALID_ARG, "node out of range");
    const cudaError_t e = launch_encode_indices(*c, node, static_cast<unsigned char *>(stream_out), (int64_t)capacity,
                                                reinterpret_cast<unsigned long long *>(sizes_out));
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_encode_indices");
    return LGC_OK;
}

lgc_status lgc_encode_innovation_positions(lgc_ctx *c, int32_t node, void *stream_out, size_t capacity, uint64_t *sizes_out)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (c->cfg.variant != LGC_VARIANT_PS) return fail(c, LGC_ERR_UNSUPPORTED, "only the parameter-server variant has innovations");
    if (!stream_out || !sizes_out || capacity < 4 || capacity % 4 != 0 || (reinterpret_cast<uintptr_t>(stream_out) & 3) != 0 ||
        (reinterpret_cast<uintptr_t>(sizes_out) & 7) != 0)
        return fail(c, LGC_ERR_INVALID_ARG, "lgc_encode_innovation_positions: buffers must be non-NULL, the stream 4-byte aligned with a capacity that is a multiple of 4");
    if (c->stage != Ctx::kCombined)
        return fail(c, LGC_ERR_BAD_STATE, "lgc_encode_innovation_positions needs the innovations of this step's lgc_combine");
    if (node < 0 || node >= c->K) return fail(c, LGC_ERR_INVALID_ARG, "node out of range");
    const cudaError_t e = launch_encode_innovation_positions(*c, node, static_cast<unsigned char *>(stream_out), (int64_t)capacity,
                                                             reinterpret_cast<unsigned long long *>(sizes_out));
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_encode_innovation_positions");
    return LGC_OK;
}

lgc_status lgc_step_host(lgc_ctx *c, const float *host_grads, float *dev_grads, float *dev_update, float *host_update,
                         int32_t choice)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (!host_grads || !dev_grads || !dev_update || !host_update) return fail(c, LGC_ERR_INVALID_ARG, "NULL buffer");
    if (!aligned16(dev_grads) || !aligned16(dev_update))
        return fail(c, LGC_ERR_INVALID_ARG, "dev_grads and dev_update must be 16-byte aligned");
    if (choice < 0 || choice >= c->K) return fail(c, LGC_ERR_INVALID_ARG, "choice (leader / common node) out of range");
    if (c->stage != Ctx::kIdle) return fail(c, LGC_ERR_BAD_STATE, "lgc_step_host must open a step");
    if (c->cfg.grad_row_stride != 0 && c->cfg.grad_row_stride != c->N)
        return fail(c, LGC_ERR_UNSUPPORTED, "lgc_step_host copies rows that are back to back: grad_row_stride must be 0 or N");
    cudaError_t e = cudaSuccess;
    if (!c->upload_stream) {
        e = cudaStreamCreateWithFlags(&c->upload_stream, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->tail_done, cudaEventDisableTiming);
        for (int k = 0; e == cudaSuccess && k < c->K; ++k) {
            cudaEvent_t ev = nullptr;
            e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
            if (e == cudaSuccess) c->row_uploaded.push_back(ev);
        }
        if (e != cudaSuccess) return cuda_fail(c, e, "lgc_step_host (streams)");
    }
    // The upload may begin once everything queued on the context's stream up to the previous call's
    // scatter has run (that call's download may still be on the bus: the two directions overlap).
    if (!c->tail_recorded) e = cudaEventRecord(c->tail_done, c->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(c->upload_stream, c->tail_done, 0);
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_step_host (order)");
    bool fused;
    lgc_status st = open_step(c, dev_grads, choice, &fused);
    if (st != LGC_OK) return st;
    // node by node: row k is accumulated while rows k+1.. are still being uploaded
    const size_t row_bytes = (size_t)c->N * sizeof(float);
    const bool by_rows = c->N % 4 == 0;           // rows of dev_grads, u and v then start 16-byte aligned
    for (int k = 0; k < c->K; ++k) {
        e = cudaMemcpyAsync(dev_grads + (int64_t)k * c->N, host_grads + (int64_t)k * c->N, row_bytes, cudaMemcpyHostToDevice,
                            c->upload_stream);
        if (e == cudaSuccess && (by_rows || k == c->K - 1)) {
            e = cudaEventRecord(c->row_uploaded[k], c->upload_stream);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(c->stream, c->row_uploaded[k], 0);
            if (e == cudaSuccess) e = by_rows ? accumulate_nodes(c, dev_grads, choice, fused, k, k + 1)
                                              : accumulate_nodes(c, dev_grads, choice, fused, 0, c->K);
        }
        if (e != cudaSuccess) {
            c->stage = Ctx::kIdle;
            return cuda_fail(c, e, "lgc_step_host (upload)");
        }
    }
    c->stage = Ctx::kAccumulated;
    c->step_grads = dev_grads;
    st = lgc_topk(c, choice, dev_update);
    if (st == LGC_OK) st = lgc_encode(c);
    if (st == LGC_OK) st = lgc_combine(c, choice);
    if (st == LGC_OK) st = lgc_decode_scatter(c, dev_update);
    if (st != LGC_OK) {
        // a stage refused or failed (the arguments were checked above, so this is a CUDA error): the
        // step is given up, so that the context accepts a new one; the message of the stage stays
        c->stage = Ctx::kIdle;
        return st;
    }
    e = cudaEventRecord(c->tail_done, c->stream);
    c->tail_recorded = e == cudaSuccess;
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(host_update, dev_update, (size_t)c->N * sizeof(float), cudaMemcpyDeviceToHost, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_step_host (download)");
    return LGC_OK;
}

lgc_status lgc_get_layout(const lgc_ctx *c, int64_t *N, int64_t *mu, int64_t *L1, int64_t *L2, int64_t *param_count)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (N) *N = c->N;
    if (mu) *mu = c->mu;
    if (L1) *L1 = c->L1;
    if (L2) *L2 = c->L2;
    if (param_count) *param_count = c->P;
    return LGC_OK;
}

const int64_t *lgc_keep_counts(const lgc_ctx *c) { return c ? c->k_l.data() : nullptr; }

lgc_status lgc_get_slots(const lgc_ctx *c, int64_t *mu_all, const int64_t **first_slot, float **val_topk_only)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (mu_all) *mu_all = c->mu_all;
    if (first_slot) *first_slot = c->kslot.data();
    if (val_topk_only) *val_topk_only = c->val_t;
    return LGC_OK;
}

lgc_status lgc_get_buffers(const lgc_ctx *c, float **u, float **v, int32_t **idx, float **val, float **code,
                           float **combined, float **inn, float **recon)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    if (u) *u = c->u;
    if (v) *v = c->v;
    if (idx) *idx = c->idx;
    if (val) *val = c->val;
    if (code) *code = c->code;
    if (combined) *combined = c->combined;
    if (inn) *inn = c->inn;
    if (recon) *recon = c->recon;
    return LGC_OK;
}

lgc_status lgc_set_ae_params(lgc_ctx *c, const float *src, size_t count)
{
    if (!c || !src) return LGC_ERR_INVALID_ARG;
    if ((int64_t)count != c->P) return fail(c, LGC_ERR_INVALID_ARG, "parameter count does not match the configuration");
    if (count == 0) return LGC_OK;
    cudaError_t e = cudaMemcpyAsync(c->params, src, count * sizeof(float), cudaMemcpyDefault, c->stream);
    if (c->ae5) c->ae5->weights_ready = false;
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    return e == cudaSuccess ? LGC_OK : cuda_fail(c, e, "lgc_set_ae_params");
}

lgc_status lgc_get_ae_params(const lgc_ctx *c, float *dst, size_t count)
{
    if (!c || !dst) return LGC_ERR_INVALID_ARG;
    if ((int64_t)count != c->P) return LGC_ERR_INVALID_ARG;
    if (count == 0) return LGC_OK;
    cudaError_t e = cudaMemcpyAsync(dst, c->params, count * sizeof(float), cudaMemcpyDefault, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    return e == cudaSuccess ? LGC_OK : LGC_ERR_CUDA;
}

lgc_status lgc_check(lgc_ctx *c)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    int32_t word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, c->errword, sizeof word, cudaMemcpyDeviceToHost, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "lgc_check");
    if (word == 0) return LGC_OK;
    launch_zero(c->errword, 16, c->stream);
    char buf[96];
    snprintf(buf, sizeof buf, "device check 0x%X: a selection kernel found inconsistent counts", (unsigned)word);
    return fail(c, LGC_ERR_DEVICE_CHECK, buf);
}

uint64_t lgc_kernel_launches(void) { return g_kernel_launches; }

lgc_status lgc_selection_stats(lgc_ctx *c, int64_t *large_segments, int64_t *served_by_accumulation,
                               int64_t *candidates_total, int64_t *candidates_max, int64_t *finished_from_data)
{
    if (!c) return LGC_ERR_INVALID_ARG;
    const size_t n = (size_t)c->S * c->sel_v.num_large;
    std::vector<int32_t> ep(n), m(n);
    if (n) {
        cudaError_t e = cudaMemcpyAsync(ep.data(), c->sel_v.seg_path, n * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(m.data(), c->sel_v.seg_m, n * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
        if (e != cudaSuccess) return cuda_fail(c, e, "lgc_selection_stats");
    }
    int64_t served = 0, total = 0, most = 0, from_data = 0;
    for (size_t i = 0; i < n; ++i) {
        served += ep[i] == 0;
        from_data += ep[i] >= 2;
        total += m[i];
        if (m[i] > most) most = m[i];
    }
    if (large_segments) *large_segments = (int64_t)n;
    if (served_by_accumulation) *served_by_accumulation = served;
    if (candidates_total) *candidates_total = total;
    if (candidates_max) *candidates_max = most;
    if (finished_from_data) *finished_from_data = from_data;
    return LGC_OK;
}

const char *lgc_status_string(lgc_status s)
{
    switch (s) {
    case LGC_OK: return "LGC_OK";
    case LGC_ERR_INVALID_ARG: return "LGC_ERR_INVALID_ARG";
    case LGC_ERR_BAD_STATE: return "LGC_ERR_BAD_STATE";
    case LGC_ERR_WORKSPACE: return "LGC_ERR_WORKSPACE";
    case LGC_ERR_UNSUPPORTED: return "LGC_ERR_UNSUPPORTED";
    case LGC_ERR_CUDA: return "LGC_ERR_CUDA";
    case LGC_ERR_DEVICE_CHECK: return "LGC_ERR_DEVICE_CHECK";
    case LGC_ERR_NO_MEMORY: return "LGC_ERR_NO_MEMORY";
    }
    return "LGC_ERR_UNKNOWN";
}

const char *lgc_last_error(const lgc_ctx *c) { return c ? c->err.c_str() : g_last_error.c_str(); }

}  // extern "C"
