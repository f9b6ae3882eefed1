// C-ABI of the ECO step library: argument validation, the work-unit tables,
// per-step scalar derivation and kernel enqueueing.  Declarations and the
// full contract of every entry point are in include/eco.h.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <unordered_set>
#include <vector>

#include "../../include/eco.h"
#include "eco_launch.h"

using eco::LaunchConfig;
using eco::StepParams;
using eco::TensorDesc;

namespace {

thread_local std::string g_thread_error;

enum LaunchKind { KIND_BLOCK_FAST = 0, KIND_BLOCK_GENERIC = 1, KIND_TENSOR = 2, KIND_ROW = 3, KIND_TENSOR_STREAM = 4,
                  KIND_ROW_STREAM = 5, KIND_TENSOR_WAVE = 6, KIND_ROW_CLUSTER = 7 };

struct Launch {
    int kind;
    size_t desc_offset;   // into d_descs
    size_t unit_offset;   // into d_unit_tensor
    uint32_t n_units;
    size_t wave_offset = 0;   // KIND_TENSOR_WAVE: into d_waves
    uint32_t n_waves = 0;
    int cluster = 1;          // KIND_ROW_CLUSTER: CTAs per cluster
};

// Options settable through eco_set_option before eco_create.
struct Options {
    int64_t l2_group_bytes = 0;    // per-tensor scale: input bytes per launch pair; -1 = half of the L2 size, 0 = one group
    int64_t reverse_pass2 = 1;     // per-tensor scale: walk pass 2 in the opposite order of pass 1
    int64_t use_stream = 1;        // 1: TMA-fed persistent kernels where the layout allows; 0: direct-load kernels only
    int64_t ctas_per_sm = 0;       // persistent grid = ctas_per_sm * SM count; 0: the kernel's own residency (2 or 3)
    int64_t fused_tensor = 2;      // per-tensor scale: both passes in one cooperative launch, wave by wave: 0 = never (launch
                                   // pair), 1 = always, 2 = when the whole context is a single wave (see eco_create)
    int64_t row_cluster = 1;       // per-row scale: 1 = rows of 33..128 segments run on thread-block clusters; 0 = one CTA per row
    int64_t wave_bytes = 100ll << 20;   // per-tensor scale, one launch: input bytes of a wave of tensors (about the L2 size)
};
Options g_options;

}  // namespace

struct eco_ctx {
    eco_config cfg;
    int device = 0;
    LaunchConfig lc{};
    std::vector<Launch> launches;
    TensorDesc* d_descs = nullptr;
    uint32_t* d_unit_tensor = nullptr;
    uint32_t* d_amax[2] = {nullptr, nullptr};
    float* d_s_old = nullptr;
    uint32_t* d_status = nullptr;
    uint32_t* d_tickets = nullptr;
    eco::WaveDesc* d_waves = nullptr;
    uint32_t* d_grid_counter = nullptr;
    uint32_t* d_wave_tickets = nullptr;   // two per wave; NULL for a single wave (static split)
    bool pending = false;          // eco_step_begin issued, eco_step_end not yet
    std::vector<TensorDesc> h_descs;      // host copy of the descriptor table (patched by eco_attach_error_buffers)
    std::vector<size_t> desc_of_tensor;   // tensor index -> its descriptor
    bool has_error_buffers = false;
    StepParams pending_params{};
    size_t n_tensors = 0;
    int grid_cap = 296;
    uint64_t calls = 0;
    bool reverse_pass2 = true;
    int num_launches = 0;
    std::string err;
};

namespace {

eco_status fail(eco_ctx* ctx, eco_status st, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_thread_error = buf;
    if (ctx) ctx->err = buf;
    return st;
}

#define ECO_CUDA(ctx, call)                                                                        \
    do {                                                                                           \
        cudaError_t e_ = (call);                                                                   \
        if (e_ != cudaSuccess)                                                                     \
            return fail(ctx, e_ == cudaErrorMemoryAllocation ? ECO_ERR_NOMEM : ECO_ERR_CUDA,       \
                        "%s failed: %s", #call, cudaGetErrorString(e_));                           \
    } while (0)

eco_status check_config(const eco_config* cfg, bool need_optimizer) {
    if (!cfg) return fail(nullptr, ECO_ERR_INVALID_ARG, "cfg is NULL");
    if (cfg->format != ECO_FORMAT_FP8_E4M3 && cfg->format != ECO_FORMAT_INT4 && cfg->format != ECO_FORMAT_FP8_E5M2)
        return fail(nullptr, ECO_ERR_UNSUPPORTED, "unknown format %d", cfg->format);
    if (cfg->granularity < ECO_SCALE_PER_TENSOR || cfg->granularity > ECO_SCALE_PER_BLOCK)
        return fail(nullptr, ECO_ERR_UNSUPPORTED, "unknown granularity %d", cfg->granularity);
    if (cfg->granularity == ECO_SCALE_PER_BLOCK && cfg->block != 128 && cfg->block != 32)
        return fail(nullptr, ECO_ERR_UNSUPPORTED, "block %d: 128 and 32 are built", cfg->block);
    if (cfg->scale_dtype != ECO_SCALE_F32 && cfg->scale_dtype != ECO_SCALE_BF16 && cfg->scale_dtype != ECO_SCALE_E8M0)
        return fail(nullptr, ECO_ERR_UNSUPPORTED, "unknown scale_dtype %d", cfg->scale_dtype);
    if (cfg->rounding != ECO_ROUND_NEAREST && cfg->rounding != ECO_ROUND_STOCHASTIC)
        return fail(nullptr, ECO_ERR_UNSUPPORTED, "unknown rounding %d", cfg->rounding);
    if (need_optimizer) {
        if (cfg->optimizer != ECO_OPT_SGDM && cfg->optimizer != ECO_OPT_ADAM)
            return fail(nullptr, ECO_ERR_UNSUPPORTED, "unknown optimizer %d", cfg->optimizer);
        if (cfg->injection != ECO_INJECT_NONE && cfg->injection != ECO_INJECT_ECO && cfg->injection != ECO_INJECT_EXACT)
            return fail(nullptr, ECO_ERR_UNSUPPORTED, "unknown injection %d", cfg->injection);
        if (cfg->injection == ECO_INJECT_EXACT && cfg->optimizer != ECO_OPT_SGDM)
            return fail(nullptr, ECO_ERR_UNSUPPORTED, "ECO_INJECT_EXACT (Appendix A) is defined for momentum SGD only");
    }
    if (cfg->reserved != 0) return fail(nullptr, ECO_ERR_INVALID_ARG, "cfg->reserved must be 0");
    return ECO_OK;
}

LaunchConfig launch_config(const eco_config& cfg) {
    LaunchConfig lc;
    lc.sm_count = 0;
    lc.format = cfg.format == ECO_FORMAT_FP8_E4M3 ? eco::FMT_FP8 : (cfg.format == ECO_FORMAT_FP8_E5M2 ? eco::FMT_E5M2 : eco::FMT_INT4);
    lc.optimizer = cfg.optimizer == ECO_OPT_ADAM ? eco::OPT_ADAM : eco::OPT_SGDM;
    lc.rounding = cfg.rounding == ECO_ROUND_STOCHASTIC ? eco::RND_SR : eco::RND_RTN;
    lc.scale_kind = cfg.scale_dtype == ECO_SCALE_BF16 ? eco::SCALE_KIND_BF16
                    : (cfg.scale_dtype == ECO_SCALE_E8M0 ? eco::SCALE_KIND_E8M0 : eco::SCALE_KIND_F32);
    lc.sub = (cfg.granularity == ECO_SCALE_PER_BLOCK && cfg.block == 32) ? 4 : 1;
    return lc;
}

uint64_t n_scales(const eco_config& cfg, int64_t rows, int64_t cols) {
    if (cfg.granularity == ECO_SCALE_PER_TENSOR) return 1;
    if (cfg.granularity == ECO_SCALE_PER_ROW) return static_cast<uint64_t>(rows);
    return static_cast<uint64_t>(rows) * static_cast<uint64_t>((cols + cfg.block - 1) / cfg.block);
}

uint64_t code_bytes(const eco_config& cfg, uint64_t numel) {
    return cfg.format == ECO_FORMAT_INT4 ? (numel + 1) / 2 : numel;
}

uint64_t scale_bytes(const eco_config& cfg, int64_t rows, int64_t cols) {
    return n_scales(cfg, rows, cols) * (cfg.scale_dtype == ECO_SCALE_BF16 ? 2 : (cfg.scale_dtype == ECO_SCALE_E8M0 ? 1 : 4));
}

eco_status check_shape(const eco_config& cfg, int64_t rows, int64_t cols, size_t i) {
    if (rows < 1 || cols < 1) return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: rows and cols must be >= 1", i);
    if (rows >= (int64_t(1) << 34) || cols >= (int64_t(1) << 32) ||
        static_cast<unsigned __int128>(rows) * static_cast<unsigned __int128>(cols) >= (static_cast<unsigned __int128>(1) << 34))
        return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: rows*cols must be < 2^34 and cols < 2^32", i);
    if (cfg.format == ECO_FORMAT_INT4 && (cols & 1))
        return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: INT4 needs an even number of columns", i);
    return ECO_OK;
}

eco_status check_device_ptr(const void* p, int device, const char* what, size_t i, bool on_device) {
    if (!p) return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: %s is NULL", i, what);
    if (reinterpret_cast<uintptr_t>(p) & 15) return fail(nullptr, ECO_ERR_ALIGNMENT, "tensor %zu: %s is not 16-byte aligned", i, what);
    if (on_device) {
        cudaPointerAttributes attr;
        cudaError_t e = cudaPointerGetAttributes(&attr, p);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return fail(nullptr, ECO_ERR_CUDA, "cudaPointerGetAttributes(%s of tensor %zu): %s", what, i, cudaGetErrorString(e));
        }
        if (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged)
            return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: %s is not device memory", i, what);
        if (attr.type == cudaMemoryTypeDevice && attr.device != device)
            return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: %s lives on device %d, context is on %d", i, what, attr.device, device);
    }
    return ECO_OK;
}

eco_status check_hyper(eco_ctx* ctx, const eco_config& cfg, float lr, float beta1, float beta2, float eps, uint64_t step) {
    if (!(lr > 0.0f) || !std::isfinite(lr)) return fail(ctx, ECO_ERR_INVALID_ARG, "lr must be finite and > 0 (got %g)", lr);
    if (!(beta1 > 0.0f && beta1 < 1.0f)) return fail(ctx, ECO_ERR_INVALID_ARG, "beta1 must be in (0,1) (got %g)", beta1);
    if (step < 1) return fail(ctx, ECO_ERR_INVALID_ARG, "step is 1-based");
    if (cfg.optimizer == ECO_OPT_ADAM) {
        if (!(beta2 > 0.0f && beta2 < 1.0f)) return fail(ctx, ECO_ERR_INVALID_ARG, "beta2 must be in (0,1) (got %g)", beta2);
        if (!(eps >= 0.0f) || !std::isfinite(eps)) return fail(ctx, ECO_ERR_INVALID_ARG, "eps must be finite and >= 0 (got %g)", eps);
    }
    return ECO_OK;
}

// Scalars of one step, each derived in binary64 from the binary32 arguments and cast once.
StepParams derive_params(const eco_config& cfg, float lr_f, float beta1_f, float beta2_f, float eps_f,
                         uint64_t step, uint64_t seed, float weight_decay_f = 0.0f, float grad_scale_f = 1.0f) {
    const double lr = lr_f, b1 = beta1_f, b2 = beta2_f;
    const double t = static_cast<double>(step);
    StepParams P;
    std::memset(&P, 0, sizeof P);
    P.beta1 = beta1_f;
    P.beta2 = beta2_f;
    P.eps = eps_f;
    P.neg_eps = -eps_f;
    P.one_minus_beta1 = static_cast<float>(1.0 - b1);
    P.one_minus_beta2 = static_cast<float>(1.0 - b2);
    P.neg_lr = -lr_f;
    P.neg_lr_wd = static_cast<float>(-(lr * static_cast<double>(weight_decay_f)));
    P.grad_scale = grad_scale_f;
    P.has_decay = weight_decay_f != 0.0f ? 1 : 0;
    P.has_grad_scale = grad_scale_f != 1.0f ? 1 : 0;
    P.fast_ok = (eps_f >= 0.0f && eps_f <= 1073741824.0f) ? 1 : 0;
    P.alpha = static_cast<float>((1.0 / lr) * (1.0 - 1.0 / b1));
    if (cfg.optimizer == ECO_OPT_ADAM) {
        const double bc1 = 1.0 - std::pow(b1, t);
        const double bc2 = 1.0 - std::pow(b2, t);
        P.inv_bc2 = static_cast<float>(1.0 / bc2);
        P.lr_over_bc1 = static_cast<float>(lr / bc1);
        P.neg_lr_over_bc1 = -P.lr_over_bc1;
        P.neg_inv_bc2 = -P.inv_bc2;
        P.adam_coef = static_cast<float>((bc1 / lr) * (1.0 - 1.0 / b1));
        // region of the fast square root / quotient as bounds on v~ and |m~| (see StepParams), 2^-20 inside
        const double in = 1.0 + std::ldexp(1.0, -20), out = 1.0 - std::ldexp(1.0, -20);
        P.fast_v_lo = static_cast<float>(std::ldexp(1.0, -80) / static_cast<double>(P.inv_bc2) * in);
        P.fast_v_hi = static_cast<float>(std::ldexp(1.0, 60) / static_cast<double>(P.inv_bc2) * out);
        P.fast_m_lo = static_cast<float>(std::ldexp(1.0, -60) / static_cast<double>(P.lr_over_bc1) * in);
        P.fast_m_hi = static_cast<float>(std::ldexp(1.0, 60) / static_cast<double>(P.lr_over_bc1) * out);
        for (float b : {P.fast_v_lo, P.fast_v_hi, P.fast_m_lo, P.fast_m_hi})
            if (!std::isnormal(b)) P.fast_ok = 0;
    }
    P.seed_lo = static_cast<uint32_t>(seed);
    P.seed_hi = static_cast<uint32_t>(seed >> 32);
    P.step_lo = static_cast<uint32_t>(step);
    P.step_hi = static_cast<uint32_t>(step >> 32);
    P.exact_qs = cfg.scale_dtype != ECO_SCALE_F32 ? 1 : 0;
    P.inject = cfg.injection == ECO_INJECT_ECO ? 1 : (cfg.injection == ECO_INJECT_EXACT ? 2 : 0);
    P.inv_lr = static_cast<float>(1.0 / lr);
    P.inv_lr_beta = static_cast<float>(1.0 / (lr * b1));
    for (uint32_t r = 0; r < 10; ++r) {
        P.rk0[r] = P.seed_lo + r * 0x9E3779B9u;
        P.rk1[r] = P.seed_hi + r * 0xBB67AE85u;
    }
    return P;
}

struct Interval {
    uintptr_t lo, hi;
    size_t tensor;
    const char* what;
};

}  // namespace

extern "C" {

const char* eco_version(void) { return "0.1.0"; }

const char* eco_last_error(const eco_ctx* ctx) { return ctx ? ctx->err.c_str() : g_thread_error.c_str(); }

eco_status eco_set_option(const char* name, int64_t value) {
    if (!name) return fail(nullptr, ECO_ERR_INVALID_ARG, "option name is NULL");
    if (!std::strcmp(name, "l2_group_bytes")) { g_options.l2_group_bytes = value; return ECO_OK; }
    if (!std::strcmp(name, "reverse_pass2")) { g_options.reverse_pass2 = value; return ECO_OK; }
    if (!std::strcmp(name, "use_stream")) { g_options.use_stream = value; return ECO_OK; }
    if (!std::strcmp(name, "fused_tensor")) { g_options.fused_tensor = value; return ECO_OK; }
    if (!std::strcmp(name, "row_cluster")) { g_options.row_cluster = value; return ECO_OK; }
    if (!std::strcmp(name, "wave_bytes")) {
        if (value < (1 << 20)) return fail(nullptr, ECO_ERR_INVALID_ARG, "wave_bytes must be at least 1 MiB");
        g_options.wave_bytes = value;
        return ECO_OK;
    }
    if (!std::strcmp(name, "ctas_per_sm")) {
        if (value < 0 || value > 3) return fail(nullptr, ECO_ERR_INVALID_ARG, "ctas_per_sm must be 0 (automatic), 1, 2 or 3");
        g_options.ctas_per_sm = value;
        return ECO_OK;
    }
    return fail(nullptr, ECO_ERR_INVALID_ARG, "unknown option '%s'", name);
}

int eco_num_launches(const eco_ctx* ctx) { return ctx ? ctx->num_launches : 0; }

eco_status eco_create(eco_ctx** out, const eco_config* cfg, const eco_tensor* tensors, size_t n, int device) {
    if (!out) return fail(nullptr, ECO_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (eco_status st = check_config(cfg, true)) return st;
    if (!tensors || n == 0) return fail(nullptr, ECO_ERR_INVALID_ARG, "empty tensor list");
    if (n > 0x7FFFFFFFu) return fail(nullptr, ECO_ERR_INVALID_ARG, "too many tensors");
    for (size_t i = 0; i < n; ++i)                       // what needs no device is refused before any CUDA call
        if (eco_status st = check_shape(*cfg, tensors[i].rows, tensors[i].cols, i)) return st;
    ECO_CUDA(nullptr, cudaSetDevice(device));
    cudaDeviceProp prop;
    ECO_CUDA(nullptr, cudaGetDeviceProperties(&prop, device));
    if (prop.major < 10) return fail(nullptr, ECO_ERR_UNSUPPORTED, "device %d is sm_%d%d; this library is built for sm_100a", device, prop.major, prop.minor);

    const bool adam = cfg->optimizer == ECO_OPT_ADAM;
    std::unordered_set<uint32_t> ids;
    std::vector<Interval> iv;
    iv.reserve(n * 5);
    for (size_t i = 0; i < n; ++i) {
        const eco_tensor& t = tensors[i];
        if (eco_status st = check_shape(*cfg, t.rows, t.cols, i)) return st;
        if ((static_cast<uint64_t>(t.row_offset) * static_cast<uint64_t>(t.cols)) % 4 != 0)
            return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: row_offset * cols must be a multiple of 4", i);
        if (static_cast<unsigned __int128>(static_cast<uint64_t>(t.row_offset) + static_cast<uint64_t>(t.rows)) *
                static_cast<unsigned __int128>(t.cols) >= (static_cast<unsigned __int128>(1) << 34))
            return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: (row_offset + rows) * cols must be < 2^34", i);
        if (!ids.insert(t.tensor_id).second) return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: duplicate tensor_id %u", i, t.tensor_id);
        if (adam && !t.v) return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: Adam needs v", i);
        if (!adam && t.v) return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: v must be NULL for SGDM", i);
        const uint64_t numel = static_cast<uint64_t>(t.rows) * static_cast<uint64_t>(t.cols);
        const struct { const void* p; uint64_t bytes; const char* what; } bufs[5] = {
            {t.w, code_bytes(*cfg, numel), "w"}, {t.scale, scale_bytes(*cfg, t.rows, t.cols), "scale"},
            {t.grad, numel * 2, "grad"}, {t.m, numel * 4, "m"}, {t.v, numel * 4, "v"}};
        for (int b = 0; b < (adam ? 5 : 4); ++b) {
            if (eco_status st = check_device_ptr(bufs[b].p, device, bufs[b].what, i, true)) return st;
            const uintptr_t lo = reinterpret_cast<uintptr_t>(bufs[b].p);
            iv.push_back({lo, lo + bufs[b].bytes, i, bufs[b].what});
        }
    }
    std::sort(iv.begin(), iv.end(), [](const Interval& a, const Interval& b) { return a.lo < b.lo; });
    for (size_t k = 1; k < iv.size(); ++k)
        if (iv[k].lo < iv[k - 1].hi)
            return fail(nullptr, ECO_ERR_INVALID_ARG, "buffers overlap: %s of tensor %zu and %s of tensor %zu",
                        iv[k - 1].what, iv[k - 1].tensor, iv[k].what, iv[k].tensor);

    eco_ctx* ctx = new (std::nothrow) eco_ctx;
    if (!ctx) return fail(nullptr, ECO_ERR_NOMEM, "out of host memory");
    ctx->cfg = *cfg;
    ctx->device = device;
    ctx->n_tensors = n;
    ctx->lc = launch_config(*cfg);
    ctx->reverse_pass2 = g_options.reverse_pass2 != 0;
    ctx->grid_cap = static_cast<int>(g_options.ctas_per_sm) * prop.multiProcessorCount;
    ctx->lc.sm_count = prop.multiProcessorCount;
    // the streaming kernels take 1x32 blocks with power-of-two scales (the microscaling layout) and every other
    // granularity with f32 / bf16 scales; the remaining combinations run on the direct-load kernels
    const bool use_stream = g_options.use_stream != 0 && ((ctx->lc.scale_kind == eco::SCALE_KIND_E8M0) == (ctx->lc.sub == 4));

    ctx->desc_of_tensor.assign(n, 0);
    // ---- work-unit tables -------------------------------------------------
    const uint64_t rpu = static_cast<uint64_t>(eco::rows_per_unit());
    std::vector<TensorDesc> descs;
    std::vector<uint32_t> unit_tensor;
    std::vector<eco::WaveDesc> waves;
    int coop_attr = 0;
    cudaDeviceGetAttribute(&coop_attr, cudaDevAttrCooperativeLaunch, device);
    const bool cooperative = coop_attr != 0;
    auto base_desc = [&](size_t i) {
        const eco_tensor& t = tensors[i];
        TensorDesc d;
        std::memset(&d, 0, sizeof d);
        d.w = static_cast<uint8_t*>(t.w);
        d.scale = t.scale;
        d.grad = static_cast<const uint16_t*>(t.grad);
        d.m = t.m;
        d.v = t.v;
        d.numel = static_cast<uint64_t>(t.rows) * static_cast<uint64_t>(t.cols);
        d.cols = static_cast<uint32_t>(t.cols);
        d.blocks_per_row = static_cast<uint32_t>((t.cols + 127) / 128);
        d.scales_per_row = cfg->granularity == ECO_SCALE_PER_BLOCK ? static_cast<uint32_t>((t.cols + cfg->block - 1) / cfg->block) : 1u;
        d.tensor_id = t.tensor_id;
        d.slot = static_cast<uint32_t>(i);
        d.index_base = static_cast<uint64_t>(t.row_offset) * static_cast<uint64_t>(t.cols);
        return d;
    };
    // Appends one launch over the tensors `members`; returns false if the grid would overflow.
    auto add_launch = [&](int kind, const std::vector<size_t>& members) -> bool {
        if (members.empty()) return true;
        Launch L;
        L.kind = kind;
        L.desc_offset = descs.size();
        L.unit_offset = unit_tensor.size();
        uint64_t units = 0;
        for (size_t k = 0; k < members.size(); ++k) {
            TensorDesc d = base_desc(members[k]);
            uint64_t nu;
            if (kind == KIND_ROW) {
                d.n_blocks = static_cast<uint64_t>(tensors[members[k]].rows);
                nu = d.n_blocks;
            } else if (kind == KIND_ROW_CLUSTER) {
                // one unit per matrix row; the CTAs of a cluster share its segments
                d.n_blocks = static_cast<uint64_t>(tensors[members[k]].rows) * d.blocks_per_row;
                nu = static_cast<uint64_t>(tensors[members[k]].rows);
            } else if (kind == KIND_ROW_STREAM) {
                // a unit is as many whole matrix rows as fit 32 rows of 128 elements
                d.n_blocks = static_cast<uint64_t>(tensors[members[k]].rows) * d.blocks_per_row;
                d.unit_rows = (static_cast<uint32_t>(eco::stream_unit_rows()) / d.blocks_per_row) * d.blocks_per_row;
                nu = (d.n_blocks + d.unit_rows - 1) / d.unit_rows;
            } else {
                d.n_blocks = (kind == KIND_TENSOR || kind == KIND_TENSOR_STREAM || kind == KIND_TENSOR_WAVE) ? (d.numel + 127) / 128
                                                   : static_cast<uint64_t>(tensors[members[k]].rows) * d.blocks_per_row;
                nu = (d.n_blocks + rpu - 1) / rpu;
            }
            if (units + nu > 0x7FFFFFFFull) return false;
            d.first_unit = static_cast<uint32_t>(units);
            ctx->desc_of_tensor[members[k]] = descs.size();
            descs.push_back(d);
            unit_tensor.insert(unit_tensor.end(), static_cast<size_t>(nu), static_cast<uint32_t>(k));
            units += nu;
        }
        L.n_units = static_cast<uint32_t>(units);
        ctx->launches.push_back(L);
        return true;
    };

    double context_in_bytes = 0;      // input bytes of one step over the whole context
    for (size_t i = 0; i < n; ++i)
        context_in_bytes += ((cfg->format == ECO_FORMAT_INT4 ? 0.5 : 1.0) + 2.0 + (adam ? 8.0 : 4.0)) *
                            static_cast<double>(tensors[i].rows) * static_cast<double>(tensors[i].cols);
    bool ok = true;
    if (cfg->granularity == ECO_SCALE_PER_BLOCK) {
        std::vector<size_t> fast, generic;
        for (size_t i = 0; i < n; ++i) ((use_stream && tensors[i].cols % 128 == 0) ? fast : generic).push_back(i);
        ok = add_launch(KIND_BLOCK_FAST, fast) && add_launch(KIND_BLOCK_GENERIC, generic);
        ctx->num_launches = static_cast<int>(ctx->launches.size());
    } else if (cfg->granularity == ECO_SCALE_PER_ROW) {
        // Matrix rows made of whole 128-element segments go to the streaming kernel: up to 32 segments as whole rows
        // per unit, up to 32 * 4 segments with a thread-block cluster of 2..4 CTAs per matrix row (one launch per
        // cluster size); anything else to the one-CTA-per-row kernel.
        std::vector<size_t> fast, generic, clustered[5];
        const int64_t seg_max = eco::stream_unit_rows();
        for (size_t i = 0; i < n; ++i) {
            const int64_t segs = tensors[i].cols / 128;
            if (!use_stream || tensors[i].cols % 128 != 0 || segs > seg_max * eco::stream_max_cluster()) generic.push_back(i);
            else if (segs <= seg_max) fast.push_back(i);
            else if (g_options.row_cluster == 0) generic.push_back(i);
            else clustered[(segs + seg_max - 1) / seg_max].push_back(i);
        }
        ok = add_launch(KIND_ROW_STREAM, fast);
        for (int c = 2; c <= eco::stream_max_cluster() && ok; ++c) {
            ok = add_launch(KIND_ROW_CLUSTER, clustered[c]);
            if (ok && !clustered[c].empty()) ctx->launches.back().cluster = c;
        }
        ok = ok && add_launch(KIND_ROW, generic);
        ctx->num_launches = static_cast<int>(ctx->launches.size());
    } else if (use_stream && cooperative && g_options.l2_group_bytes == 0 &&
               (g_options.fused_tensor == 1 || (g_options.fused_tensor == 2 && context_in_bytes <= static_cast<double>(g_options.wave_bytes)))) {
        // Per-tensor scale, one cooperative launch: waves of whole tensors whose inputs are about as large as L2.  A
        // tensor of at least half the budget is a wave of its own; smaller ones are packed in the order given.
        // Default: only when the whole context is one wave (it then stays on the chip between the passes and the step
        // is a single launch).  On larger sets the launch pair is faster although it moves more bytes: with two front
        // halves the step is bound by instruction issue, and the grid barrier of every wave idles the SMs that arrive early.
        const double in_bytes_per_elem = (cfg->format == ECO_FORMAT_INT4 ? 0.5 : 1.0) + 2.0 + (adam ? 8.0 : 4.0);
        const double budget = static_cast<double>(g_options.wave_bytes);
        std::vector<std::vector<size_t>> groups;
        std::vector<size_t> small, generic;
        double small_bytes = 0;
        for (size_t i = 0; i < n; ++i) {
            const uint64_t numel = static_cast<uint64_t>(tensors[i].rows) * static_cast<uint64_t>(tensors[i].cols);
            if (numel % 128 != 0) { generic.push_back(i); continue; }
            const double b = in_bytes_per_elem * static_cast<double>(numel);
            if (b >= budget / 2) { groups.push_back({i}); continue; }
            if (!small.empty() && small_bytes + b > budget) {
                groups.push_back(small);
                small.clear();
                small_bytes = 0;
            }
            small.push_back(i);
            small_bytes += b;
        }
        if (!small.empty()) groups.push_back(small);
        std::vector<size_t> members;
        for (const auto& g : groups) members.insert(members.end(), g.begin(), g.end());
        ok = add_launch(KIND_TENSOR_WAVE, members);
        if (ok && !members.empty()) {
            Launch& L = ctx->launches.back();
            L.wave_offset = waves.size();
            size_t k = 0;
            for (const auto& g : groups) {
                eco::WaveDesc wd;
                wd.first_unit = descs[L.desc_offset + k].first_unit;
                const TensorDesc& last = descs[L.desc_offset + k + g.size() - 1];
                const uint32_t last_units = static_cast<uint32_t>((last.n_blocks + rpu - 1) / rpu);
                wd.n_units = last.first_unit + last_units - wd.first_unit;
                waves.push_back(wd);
                k += g.size();
            }
            L.n_waves = static_cast<uint32_t>(groups.size());
        }
        if (ok) ok = add_launch(KIND_TENSOR, generic);
        ctx->num_launches = (members.empty() ? 0 : 1) + (generic.empty() ? 0 : 2);
    } else {
        // Per-tensor scale: pass 1 + pass 2 per group of tensors whose inputs fit the L2 budget, so
        // that pass 2 finds what pass 1 read still cached.
        int64_t budget = g_options.l2_group_bytes;
        if (budget < 0) budget = static_cast<int64_t>(prop.l2CacheSize) / 2;
        const double in_bytes_per_elem = (cfg->format == ECO_FORMAT_INT4 ? 0.5 : 1.0) + 2.0 + (adam ? 8.0 : 4.0);
        std::vector<size_t> group;
        double group_bytes = 0;
        // tensors made of whole 128-element rows go to the streaming kernels, the rest to the direct-load ones
        auto flush_group = [&]() {
            std::vector<size_t> fast, generic;
            for (size_t i : group) {
                const uint64_t numel = static_cast<uint64_t>(tensors[i].rows) * static_cast<uint64_t>(tensors[i].cols);
                ((use_stream && numel % 128 == 0) ? fast : generic).push_back(i);
            }
            return add_launch(KIND_TENSOR_STREAM, fast) && add_launch(KIND_TENSOR, generic);
        };
        for (size_t i = 0; i < n && ok; ++i) {
            const double b = in_bytes_per_elem * static_cast<double>(tensors[i].rows) * static_cast<double>(tensors[i].cols);
            if (!group.empty() && budget > 0 && group_bytes + b > static_cast<double>(budget)) {
                ok = flush_group();
                group.clear();
                group_bytes = 0;
            }
            group.push_back(i);
            group_bytes += b;
        }
        if (ok) ok = flush_group();
        ctx->num_launches = 2 * static_cast<int>(ctx->launches.size());
    }
    if (!ok) {
        delete ctx;
        return fail(nullptr, ECO_ERR_UNSUPPORTED, "tensor list too large for one launch grid");
    }

    auto cleanup = [&](eco_status st) {
        eco_destroy(ctx);
        return st;
    };
#define ECO_CUDA_CTX(call)                                                                                  \
    do {                                                                                                    \
        cudaError_t e_ = (call);                                                                            \
        if (e_ != cudaSuccess)                                                                              \
            return cleanup(fail(nullptr, e_ == cudaErrorMemoryAllocation ? ECO_ERR_NOMEM : ECO_ERR_CUDA,    \
                                "%s failed: %s", #call, cudaGetErrorString(e_)));                           \
    } while (0)
    ECO_CUDA_CTX(cudaMalloc(&ctx->d_descs, descs.size() * sizeof(TensorDesc)));
    ECO_CUDA_CTX(cudaMalloc(&ctx->d_unit_tensor, std::max<size_t>(unit_tensor.size(), 1) * sizeof(uint32_t)));
    ECO_CUDA_CTX(cudaMemcpy(ctx->d_descs, descs.data(), descs.size() * sizeof(TensorDesc), cudaMemcpyHostToDevice));
    ctx->h_descs = descs;
    ECO_CUDA_CTX(cudaMemcpy(ctx->d_unit_tensor, unit_tensor.data(), unit_tensor.size() * sizeof(uint32_t), cudaMemcpyHostToDevice));
    if (cfg->granularity == ECO_SCALE_PER_TENSOR) {
        for (int p = 0; p < 2; ++p) {
            ECO_CUDA_CTX(cudaMalloc(&ctx->d_amax[p], n * sizeof(uint32_t)));
            ECO_CUDA_CTX(cudaMemset(ctx->d_amax[p], 0, n * sizeof(uint32_t)));
        }
        ECO_CUDA_CTX(cudaMalloc(&ctx->d_s_old, n * sizeof(float)));
    }
    ECO_CUDA_CTX(cudaMalloc(&ctx->d_status, sizeof(uint32_t)));
    ECO_CUDA_CTX(cudaMemset(ctx->d_status, 0, sizeof(uint32_t)));
    ECO_CUDA_CTX(cudaMalloc(&ctx->d_tickets, 2 * sizeof(uint32_t)));
    ECO_CUDA_CTX(cudaMemset(ctx->d_tickets, 0, 2 * sizeof(uint32_t)));
    if (!waves.empty()) {
        ECO_CUDA_CTX(cudaMalloc(&ctx->d_waves, waves.size() * sizeof(eco::WaveDesc)));
        ECO_CUDA_CTX(cudaMemcpy(ctx->d_waves, waves.data(), waves.size() * sizeof(eco::WaveDesc), cudaMemcpyHostToDevice));
        ECO_CUDA_CTX(cudaMalloc(&ctx->d_grid_counter, 2 * sizeof(uint32_t)));
        ECO_CUDA_CTX(cudaMemset(ctx->d_grid_counter, 0, 2 * sizeof(uint32_t)));
        if (waves.size() > 1) {
            ECO_CUDA_CTX(cudaMalloc(&ctx->d_wave_tickets, 2 * waves.size() * sizeof(uint32_t)));
            ECO_CUDA_CTX(cudaMemset(ctx->d_wave_tickets, 0, 2 * waves.size() * sizeof(uint32_t)));
        }
    }
    ECO_CUDA_CTX(cudaDeviceSynchronize());
#undef ECO_CUDA_CTX
    *out = ctx;
    return ECO_OK;
}

}  // extern "C"

namespace {
enum { PASS_BOTH = 0, PASS_AMAX = 1, PASS_APPLY = 2 };
eco_status enqueue_step(eco_ctx* ctx, const StepParams& P, void* cuda_stream, int pass = PASS_BOTH);
}

extern "C" {

eco_status eco_step(eco_ctx* ctx, float lr, float beta1, float beta2, float eps,
                    uint64_t step, uint64_t seed, void* cuda_stream) {
    if (!ctx) return fail(nullptr, ECO_ERR_INVALID_ARG, "ctx is NULL");
    if (eco_status st = check_hyper(ctx, ctx->cfg, lr, beta1, beta2, eps, step)) return st;
    return enqueue_step(ctx, derive_params(ctx->cfg, lr, beta1, beta2, eps, step, seed), cuda_stream);
}

eco_status eco_step_ex(eco_ctx* ctx, const eco_hyper* h, void* cuda_stream) {
    if (!ctx) return fail(nullptr, ECO_ERR_INVALID_ARG, "ctx is NULL");
    if (!h) return fail(ctx, ECO_ERR_INVALID_ARG, "hyper is NULL");
    if (h->reserved != 0) return fail(ctx, ECO_ERR_INVALID_ARG, "hyper->reserved must be 0");
    if (eco_status st = check_hyper(ctx, ctx->cfg, h->lr, h->beta1, h->beta2, h->eps, h->step)) return st;
    if (!(h->weight_decay >= 0.0f) || !std::isfinite(h->weight_decay))
        return fail(ctx, ECO_ERR_INVALID_ARG, "weight_decay must be finite and >= 0 (got %g)", h->weight_decay);
    if (!std::isfinite(h->grad_scale)) return fail(ctx, ECO_ERR_INVALID_ARG, "grad_scale must be finite (got %g)", h->grad_scale);
    return enqueue_step(ctx, derive_params(ctx->cfg, h->lr, h->beta1, h->beta2, h->eps, h->step, h->seed,
                                           h->weight_decay, h->grad_scale), cuda_stream);
}

eco_status eco_step_begin(eco_ctx* ctx, const eco_hyper* h, void* cuda_stream) {
    if (!ctx) return fail(nullptr, ECO_ERR_INVALID_ARG, "ctx is NULL");
    if (ctx->cfg.granularity != ECO_SCALE_PER_TENSOR)
        return fail(ctx, ECO_ERR_UNSUPPORTED, "eco_step_begin / eco_step_end are for ECO_SCALE_PER_TENSOR; other granularities need no exchange");
    if (!h) return fail(ctx, ECO_ERR_INVALID_ARG, "hyper is NULL");
    if (h->reserved != 0) return fail(ctx, ECO_ERR_INVALID_ARG, "hyper->reserved must be 0");
    if (eco_status st = check_hyper(ctx, ctx->cfg, h->lr, h->beta1, h->beta2, h->eps, h->step)) return st;
    if (!(h->weight_decay >= 0.0f) || !std::isfinite(h->weight_decay))
        return fail(ctx, ECO_ERR_INVALID_ARG, "weight_decay must be finite and >= 0 (got %g)", h->weight_decay);
    if (!std::isfinite(h->grad_scale)) return fail(ctx, ECO_ERR_INVALID_ARG, "grad_scale must be finite (got %g)", h->grad_scale);
    const StepParams P = derive_params(ctx->cfg, h->lr, h->beta1, h->beta2, h->eps, h->step, h->seed, h->weight_decay, h->grad_scale);
    if (eco_status st = enqueue_step(ctx, P, cuda_stream, PASS_AMAX)) return st;
    ctx->pending_params = P;
    ctx->pending = true;
    return ECO_OK;
}

eco_status eco_amax_buffer(eco_ctx* ctx, void** device_ptr, size_t* n) {
    if (!ctx || !device_ptr || !n) return fail(ctx, ECO_ERR_INVALID_ARG, "NULL argument");
    if (ctx->cfg.granularity != ECO_SCALE_PER_TENSOR) return fail(ctx, ECO_ERR_UNSUPPORTED, "only per-tensor scales have an amax vector");
    *device_ptr = ctx->d_amax[ctx->calls & 1];
    *n = ctx->n_tensors;
    return ECO_OK;
}

eco_status eco_step_end(eco_ctx* ctx, void* cuda_stream) {
    if (!ctx) return fail(nullptr, ECO_ERR_INVALID_ARG, "ctx is NULL");
    if (!ctx->pending) return fail(ctx, ECO_ERR_INVALID_ARG, "eco_step_end without a pending eco_step_begin");
    if (eco_status st = enqueue_step(ctx, ctx->pending_params, cuda_stream, PASS_APPLY)) return st;
    ctx->pending = false;
    return ECO_OK;
}

}  // extern "C"

namespace {

eco_status enqueue_step(eco_ctx* ctx, const StepParams& P, void* cuda_stream, int pass) {
    if (P.inject == 2 && !ctx->has_error_buffers)
        return fail(ctx, ECO_ERR_INVALID_ARG, "ECO_INJECT_EXACT needs eco_attach_error_buffers first");
    if (ctx->pending && pass != PASS_APPLY)
        return fail(ctx, ECO_ERR_INVALID_ARG, "eco_step_begin is pending: call eco_step_end first");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int parity = static_cast<int>(ctx->calls & 1);
    for (const Launch& L : ctx->launches) {
        const TensorDesc* descs = ctx->d_descs + L.desc_offset;
        const uint32_t* units = ctx->d_unit_tensor + L.unit_offset;
        switch (L.kind) {
            case KIND_BLOCK_FAST:
                ECO_CUDA(ctx, eco::launch_stream(ctx->lc, ctx->lc.sub == 4 ? eco::STREAM_BLOCK32 : eco::STREAM_BLOCK, descs, units, L.n_units, P, nullptr, nullptr,
                                                 nullptr, false, ctx->d_tickets, ctx->d_status, ctx->grid_cap, stream, ctx->has_error_buffers));
                break;
            case KIND_BLOCK_GENERIC:
                ECO_CUDA(ctx, eco::launch_block128(ctx->lc, descs, units, L.n_units, true, P, stream));
                break;
            case KIND_TENSOR_STREAM:
                if (pass != PASS_APPLY)
                    ECO_CUDA(ctx, eco::launch_stream(ctx->lc, eco::STREAM_TENSOR_AMAX, descs, units, L.n_units, P,
                                                     ctx->d_amax[parity], nullptr, ctx->d_s_old, false, ctx->d_tickets,
                                                     ctx->d_status, ctx->grid_cap, stream));
                if (pass != PASS_AMAX)
                    ECO_CUDA(ctx, eco::launch_stream(ctx->lc, eco::STREAM_TENSOR_APPLY, descs, units, L.n_units, P,
                                                     ctx->d_amax[parity], ctx->d_amax[parity ^ 1], ctx->d_s_old,
                                                     ctx->reverse_pass2, ctx->d_tickets, ctx->d_status, ctx->grid_cap, stream, ctx->has_error_buffers));
                break;
            case KIND_TENSOR_WAVE:
                if (pass == PASS_BOTH) {
                    ECO_CUDA(ctx, eco::launch_wave(ctx->lc, descs, units, ctx->d_waves + L.wave_offset, L.n_waves, P,
                                                   ctx->d_amax[parity], ctx->d_amax[parity ^ 1], ctx->d_s_old,
                                                   ctx->d_grid_counter,
                                                   ctx->d_wave_tickets ? ctx->d_wave_tickets + 2 * L.wave_offset : nullptr,
                                                   ctx->d_status, ctx->grid_cap, stream, ctx->has_error_buffers));
                    break;
                }
                // the step cut in two for an amax exchange between ranks: the two passes as separate launches
                if (pass != PASS_APPLY)
                    ECO_CUDA(ctx, eco::launch_stream(ctx->lc, eco::STREAM_TENSOR_AMAX, descs, units, L.n_units, P,
                                                     ctx->d_amax[parity], nullptr, ctx->d_s_old, false, ctx->d_tickets,
                                                     ctx->d_status, ctx->grid_cap, stream));
                if (pass != PASS_AMAX)
                    ECO_CUDA(ctx, eco::launch_stream(ctx->lc, eco::STREAM_TENSOR_APPLY, descs, units, L.n_units, P,
                                                     ctx->d_amax[parity], ctx->d_amax[parity ^ 1], ctx->d_s_old,
                                                     ctx->reverse_pass2, ctx->d_tickets, ctx->d_status, ctx->grid_cap, stream, ctx->has_error_buffers));
                break;
            case KIND_ROW:
                ECO_CUDA(ctx, eco::launch_row(ctx->lc, descs, units, L.n_units, P, stream));
                break;
            case KIND_ROW_CLUSTER:
                ECO_CUDA(ctx, eco::launch_stream(ctx->lc, eco::STREAM_ROW, descs, units, L.n_units, P, nullptr, nullptr,
                                                 nullptr, false, ctx->d_tickets, ctx->d_status, ctx->grid_cap, stream,
                                                 ctx->has_error_buffers, L.cluster));
                break;
            case KIND_ROW_STREAM:
                ECO_CUDA(ctx, eco::launch_stream(ctx->lc, eco::STREAM_ROW, descs, units, L.n_units, P, nullptr, nullptr,
                                                 nullptr, false, ctx->d_tickets, ctx->d_status, ctx->grid_cap, stream, ctx->has_error_buffers));
                break;
            case KIND_TENSOR:
                if (pass != PASS_APPLY)
                    ECO_CUDA(ctx, eco::launch_tensor_amax(ctx->lc, descs, units, L.n_units, P, ctx->d_amax[parity], ctx->d_s_old, stream));
                if (pass != PASS_AMAX)
                    ECO_CUDA(ctx, eco::launch_tensor_apply(ctx->lc, descs, units, L.n_units, P, ctx->d_amax[parity],
                                                           ctx->d_amax[parity ^ 1], ctx->d_s_old, ctx->reverse_pass2, stream));
                break;
        }
    }
    if (pass != PASS_AMAX) ctx->calls++;       // the amax slots alternate by step parity
    return ECO_OK;
}

}  // namespace

extern "C" {

eco_status eco_check(eco_ctx* ctx, void* cuda_stream) {
    if (!ctx) return fail(nullptr, ECO_ERR_INVALID_ARG, "ctx is NULL");
    ECO_CUDA(ctx, cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
    uint32_t code = 0;
    ECO_CUDA(ctx, cudaMemcpy(&code, ctx->d_status, sizeof code, cudaMemcpyDeviceToHost));
    if (code != 0)
        return fail(ctx, ECO_ERR_TIMEOUT, "a bounded wait inside a kernel expired (code %u: 1 = producer waiting for a free "
                    "stage, 2 = producer draining its copies, 3 = consumer waiting for data, 4/5 = per-row exchange, 6 = grid barrier of the "
                    "single-launch per-tensor step, 7 = self-test, 8 = consumer warps meeting, 9 = row maximum from the cluster's peers)", code);
    return ECO_OK;
}

eco_status eco_attach_error_buffers(eco_ctx* ctx, float* const* e, size_t n) {
    if (!ctx) return fail(nullptr, ECO_ERR_INVALID_ARG, "ctx is NULL");
    if (!e || n != ctx->n_tensors) return fail(ctx, ECO_ERR_INVALID_ARG, "need one error buffer per tensor of the context (%zu)", ctx->n_tensors);
    ECO_CUDA(ctx, cudaSetDevice(ctx->device));
    for (size_t i = 0; i < n; ++i) {
        if (eco_status st = check_device_ptr(e[i], ctx->device, "error buffer", i, true)) { ctx->err = g_thread_error; return st; }
    }
    for (size_t i = 0; i < n; ++i) ctx->h_descs[ctx->desc_of_tensor[i]].e = e[i];
    ECO_CUDA(ctx, cudaDeviceSynchronize());
    ECO_CUDA(ctx, cudaMemcpy(ctx->d_descs, ctx->h_descs.data(), ctx->h_descs.size() * sizeof(TensorDesc), cudaMemcpyHostToDevice));
    ctx->has_error_buffers = true;
    return ECO_OK;
}

eco_status eco_selftest_wait(eco_ctx* ctx, int64_t limit_cycles, void* cuda_stream) {
    if (!ctx) return fail(nullptr, ECO_ERR_INVALID_ARG, "ctx is NULL");
    if (limit_cycles < 1 || limit_cycles > 2000000000LL)
        return fail(ctx, ECO_ERR_INVALID_ARG, "limit_cycles must be in 1..2e9 (got %lld)", static_cast<long long>(limit_cycles));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    ECO_CUDA(ctx, eco::launch_wait_selftest(ctx->d_status, limit_cycles, stream));
    const eco_status st = eco_check(ctx, cuda_stream);
    // the status word is sticky by design; the self-test owns it for the length of the call
    ECO_CUDA(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof(uint32_t), stream));
    ECO_CUDA(ctx, cudaStreamSynchronize(stream));
    return st;
}

eco_status eco_selftest_grid_wait(eco_ctx* ctx, int64_t limit_cycles, void* cuda_stream) {
    if (!ctx) return fail(nullptr, ECO_ERR_INVALID_ARG, "ctx is NULL");
    if (limit_cycles < 1 || limit_cycles > 2000000000LL)
        return fail(ctx, ECO_ERR_INVALID_ARG, "limit_cycles must be in 1..2e9 (got %lld)", static_cast<long long>(limit_cycles));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the self-test's arrival counter: the context's ticket words, which are zero between steps (and zeroed again below)
    ECO_CUDA(ctx, cudaMemsetAsync(ctx->d_tickets, 0, 2 * sizeof(uint32_t), stream));
    ECO_CUDA(ctx, eco::launch_grid_wait_selftest(ctx->d_tickets, ctx->d_status, limit_cycles, stream));
    const eco_status st = eco_check(ctx, cuda_stream);
    ECO_CUDA(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof(uint32_t), stream));
    ECO_CUDA(ctx, cudaMemsetAsync(ctx->d_tickets, 0, 2 * sizeof(uint32_t), stream));
    ECO_CUDA(ctx, cudaStreamSynchronize(stream));
    return st;
}

eco_status eco_destroy(eco_ctx* ctx) {
    if (!ctx) return ECO_OK;
    cudaSetDevice(ctx->device);
    cudaDeviceSynchronize();
    cudaFree(ctx->d_descs);
    cudaFree(ctx->d_unit_tensor);
    cudaFree(ctx->d_amax[0]);
    cudaFree(ctx->d_amax[1]);
    cudaFree(ctx->d_s_old);
    cudaFree(ctx->d_status);
    cudaFree(ctx->d_tickets);
    cudaFree(ctx->d_waves);
    cudaFree(ctx->d_grid_counter);
    cudaFree(ctx->d_wave_tickets);
    delete ctx;
    return ECO_OK;
}

eco_status eco_quantize(const eco_config* cfg, const float* x, int64_t rows, int64_t cols,
                        void* w, void* scale, uint64_t seed, uint64_t step, uint32_t tensor_id,
                        int device, void* cuda_stream) {
    if (eco_status st = check_config(cfg, false)) return st;
    if (eco_status st = check_shape(*cfg, rows, cols, 0)) return st;
    ECO_CUDA(nullptr, cudaSetDevice(device));
    if (eco_status st = check_device_ptr(x, device, "x", 0, true)) return st;
    if (eco_status st = check_device_ptr(w, device, "w", 0, true)) return st;
    if (eco_status st = check_device_ptr(scale, device, "scale", 0, true)) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    LaunchConfig lc = launch_config(*cfg);
    eco_config c2 = *cfg;
    c2.optimizer = ECO_OPT_SGDM;
    StepParams P = derive_params(c2, 1.0f, 0.5f, 0.5f, 0.0f, step, seed);
    const uint64_t numel = static_cast<uint64_t>(rows) * static_cast<uint64_t>(cols);
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    const uint64_t cap = static_cast<uint64_t>(sms) * 16;
    if (cfg->granularity == ECO_SCALE_PER_TENSOR) {
        uint32_t* scratch = nullptr;
        ECO_CUDA(nullptr, cudaMallocAsync(&scratch, sizeof(uint32_t), stream));
        ECO_CUDA(nullptr, cudaMemsetAsync(scratch, 0, sizeof(uint32_t), stream));
        const uint32_t grid = static_cast<uint32_t>(std::min<uint64_t>(cap, (numel + 1023) / 1024));
        ECO_CUDA(nullptr, eco::launch_quantize(lc, x, static_cast<uint8_t*>(w), scale, rows, static_cast<uint32_t>(cols), 0, P, tensor_id, scratch, grid, stream));
        ECO_CUDA(nullptr, eco::launch_quantize(lc, x, static_cast<uint8_t*>(w), scale, rows, static_cast<uint32_t>(cols), 1, P, tensor_id, scratch, grid, stream));
        ECO_CUDA(nullptr, cudaFreeAsync(scratch, stream));
    } else if (cfg->granularity == ECO_SCALE_PER_ROW) {
        const uint32_t grid = static_cast<uint32_t>(std::min<uint64_t>(cap, static_cast<uint64_t>(rows)));
        ECO_CUDA(nullptr, eco::launch_quantize(lc, x, static_cast<uint8_t*>(w), scale, rows, static_cast<uint32_t>(cols), 2, P, tensor_id, nullptr, grid, stream));
    } else {
        const uint64_t n_blocks = static_cast<uint64_t>(rows) * static_cast<uint64_t>((cols + 127) / 128);
        const uint32_t grid = static_cast<uint32_t>(std::min<uint64_t>(cap, (n_blocks + 7) / 8));
        ECO_CUDA(nullptr, eco::launch_quantize(lc, x, static_cast<uint8_t*>(w), scale, rows, static_cast<uint32_t>(cols), lc.sub == 4 ? 4 : 3, P, tensor_id, nullptr, grid, stream));
    }
    return ECO_OK;
}

}  // extern "C"

// State held in HOST memory: the tensor list is cut into chunks of whole tensors (about 256 MB of state
// each) that move through three device slots.  While chunk i is stepped, chunk i+1 is copied in and chunk
// i-1 is copied out, so both directions of the host link stay busy.  Every buffer inside a slot is
// 256-byte aligned.  Each chunk has its own eco_ctx bound to the slot it will occupy.
struct eco_host_ctx {
    struct Place { uint64_t w, scale, grad, m, v, wb, sb, gb, mb; };
    struct Chunk { size_t first, count; uint64_t bytes; };
    struct Copy { void* dev; void* host; uint64_t bytes; };   // one cudaMemcpyAsync (several tensors when both sides are contiguous)
    eco_config cfg;
    int device = 0;
    bool adam = false;
    std::vector<eco_tensor> host, dev;
    std::vector<Place> place;
    std::vector<Chunk> chunks;
    std::vector<std::vector<Copy>> copies_in, copies_out;   // per chunk
    std::vector<eco_ctx*> ctxs;
    std::vector<cudaEvent_t> ev_in, ev_run, ev_out;
    cudaStream_t s_in = nullptr, s_run = nullptr, s_out = nullptr;
    uint8_t* arena = nullptr;
    uint64_t slot_bytes = 0, up = 0, down = 0;
    int n_slots = 0;
};

// True when a and b lie inside the same CUDA allocation (pinned host memory or device memory): the driver reports
// the start of the allocation a pointer belongs to.  Anything it does not know (pageable memory) is "no".
static bool same_allocation(const void* a, const void* b) {
    using Fn = int (*)(void*, int, unsigned long long);       // cuPointerGetAttribute(data, attribute, pointer)
    static Fn fn = []() -> Fn {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuPointerGetAttribute", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<Fn>(p);
    }();
    if (!fn) return false;
    constexpr int kRangeStart = 11;                             // CU_POINTER_ATTRIBUTE_RANGE_START_ADDR
    unsigned long long sa = 0, sb = 0;
    if (fn(&sa, kRangeStart, reinterpret_cast<unsigned long long>(a)) != 0) return false;
    if (fn(&sb, kRangeStart, reinterpret_cast<unsigned long long>(b)) != 0) return false;
    return sa != 0 && sa == sb;
}

extern "C" {

eco_status eco_host_destroy(eco_host_ctx* h) {
    if (!h) return ECO_OK;
    cudaSetDevice(h->device);
    for (eco_ctx* c : h->ctxs) if (c) eco_destroy(c);
    for (auto* v : {&h->ev_in, &h->ev_run, &h->ev_out}) for (cudaEvent_t e : *v) if (e) cudaEventDestroy(e);
    if (h->s_in) cudaStreamDestroy(h->s_in);
    if (h->s_run) cudaStreamDestroy(h->s_run);
    if (h->s_out) cudaStreamDestroy(h->s_out);
    cudaFree(h->arena);
    delete h;
    return ECO_OK;
}

eco_status eco_host_create(eco_host_ctx** out, const eco_config* cfg, const eco_tensor* tensors, size_t n, int device) {
    if (!out) return fail(nullptr, ECO_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (eco_status st = check_config(cfg, true)) return st;
    if (!tensors || n == 0) return fail(nullptr, ECO_ERR_INVALID_ARG, "empty tensor list");
    const bool adam = cfg->optimizer == ECO_OPT_ADAM;
    for (size_t i = 0; i < n; ++i) {
        const eco_tensor& t = tensors[i];
        if (eco_status st = check_shape(*cfg, t.rows, t.cols, i)) return st;
        if (!t.w || !t.scale || !t.grad || !t.m || (adam && !t.v) || (!adam && t.v))
            return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: NULL buffer (or v given for SGDM)", i);
    }
    ECO_CUDA(nullptr, cudaSetDevice(device));
    eco_host_ctx* h = new (std::nothrow) eco_host_ctx;
    if (!h) return fail(nullptr, ECO_ERR_NOMEM, "out of host memory");
    h->cfg = *cfg;
    h->device = device;
    h->adam = adam;
    h->host.assign(tensors, tensors + n);
    h->dev.assign(tensors, tensors + n);
    h->place.resize(n);
    auto align = [](uint64_t x) { return (x + 255) & ~uint64_t(255); };
    constexpr uint64_t kChunkTarget = 256ull << 20;
    constexpr int kSlots = 3;
    {
        // chunks: consecutive tensors up to the target size
        eco_host_ctx::Chunk c{0, 0, 0};
        for (size_t i = 0; i < n; ++i) {
            const uint64_t numel = static_cast<uint64_t>(tensors[i].rows) * static_cast<uint64_t>(tensors[i].cols);
            eco_host_ctx::Place& p = h->place[i];
            p.wb = code_bytes(*cfg, numel); p.sb = scale_bytes(*cfg, tensors[i].rows, tensors[i].cols);
            p.gb = numel * 2; p.mb = numel * 4;
            const uint64_t need = align(p.wb) + align(p.sb) + align(p.gb) + align(p.mb) * (adam ? 2 : 1);
            if (c.count > 0 && c.bytes + need > kChunkTarget) {
                h->chunks.push_back(c);
                c = eco_host_ctx::Chunk{i, 0, 0};
            }
            c.bytes += need;
            c.count++;
            h->slot_bytes = std::max(h->slot_bytes, c.bytes);
        }
        h->chunks.push_back(c);
        // inside a chunk the buffers are laid out by kind (all codes, all scales, all gradients, all m, all v), so
        // that state which is contiguous on the host is contiguous on the device too and moves in one copy
        for (const eco_host_ctx::Chunk& ch : h->chunks) {
            uint64_t region[5] = {0, 0, 0, 0, 0};
            for (size_t i = ch.first; i < ch.first + ch.count; ++i) {
                const eco_host_ctx::Place& p = h->place[i];
                region[0] += align(p.wb); region[1] += align(p.sb); region[2] += align(p.gb); region[3] += align(p.mb);
                if (adam) region[4] += align(p.mb);
            }
            uint64_t off[5] = {0, region[0], region[0] + region[1], region[0] + region[1] + region[2],
                               region[0] + region[1] + region[2] + region[3]};
            for (size_t i = ch.first; i < ch.first + ch.count; ++i) {
                eco_host_ctx::Place& p = h->place[i];
                p.w = off[0]; off[0] += align(p.wb);
                p.scale = off[1]; off[1] += align(p.sb);
                p.grad = off[2]; off[2] += align(p.gb);
                p.m = off[3]; off[3] += align(p.mb);
                p.v = off[4]; if (adam) off[4] += align(p.mb);
            }
        }
    }
    h->n_slots = static_cast<int>(std::min<size_t>(kSlots, h->chunks.size()));
    const size_t nc = h->chunks.size();
    h->ctxs.assign(nc, nullptr);
    h->ev_in.assign(nc, nullptr); h->ev_run.assign(nc, nullptr); h->ev_out.assign(nc, nullptr);
    h->copies_in.assign(nc, {});
    h->copies_out.assign(nc, {});
#define ECO_CUDA_H(call)                                                                             \
    do {                                                                                             \
        cudaError_t e_ = (call);                                                                     \
        if (e_ != cudaSuccess) {                                                                     \
            eco_status st_ = fail(nullptr, e_ == cudaErrorMemoryAllocation ? ECO_ERR_NOMEM : ECO_ERR_CUDA, \
                                  "%s failed: %s", #call, cudaGetErrorString(e_));                   \
            eco_host_destroy(h);                                                                     \
            return st_;                                                                              \
        }                                                                                            \
    } while (0)
    ECO_CUDA_H(cudaMalloc(&h->arena, h->slot_bytes * h->n_slots));
    ECO_CUDA_H(cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking));
    ECO_CUDA_H(cudaStreamCreateWithFlags(&h->s_run, cudaStreamNonBlocking));
    ECO_CUDA_H(cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking));
    for (size_t c = 0; c < nc; ++c) {
        uint8_t* base = h->arena + h->slot_bytes * (c % h->n_slots);
        for (size_t i = h->chunks[c].first; i < h->chunks[c].first + h->chunks[c].count; ++i) {
            const eco_host_ctx::Place& p = h->place[i];
            h->dev[i].w = base + p.w;
            h->dev[i].scale = base + p.scale;
            h->dev[i].grad = base + p.grad;
            h->dev[i].m = reinterpret_cast<float*>(base + p.m);
            h->dev[i].v = adam ? reinterpret_cast<float*>(base + p.v) : nullptr;
        }
        eco_status rc = eco_create(&h->ctxs[c], cfg, h->dev.data() + h->chunks[c].first, h->chunks[c].count, device);
        if (rc != ECO_OK) { eco_host_destroy(h); return rc; }
        // copy lists, kind by kind; a buffer joins the previous copy when it follows it directly on both sides and
        // the two host buffers are parts of one allocation (neighbouring addresses alone do not make one copy legal)
        auto add = [](std::vector<eco_host_ctx::Copy>& v, void* dev, const void* host, uint64_t bytes) {
            if (!v.empty() && static_cast<uint8_t*>(v.back().dev) + v.back().bytes == dev &&
                static_cast<uint8_t*>(v.back().host) + v.back().bytes == host && same_allocation(v.back().host, host))
                v.back().bytes += bytes;
            else
                v.push_back(eco_host_ctx::Copy{dev, const_cast<void*>(host), bytes});
        };
        const size_t first = h->chunks[c].first, last = first + h->chunks[c].count;
        for (int kind = 0; kind < 5; ++kind) {
            if (kind == 4 && !adam) continue;
            for (size_t i = first; i < last; ++i) {
                const eco_host_ctx::Place& p = h->place[i];
                const eco_tensor &hs = h->host[i], &dv = h->dev[i];
                void* d = kind == 0 ? dv.w : kind == 1 ? dv.scale : kind == 2 ? const_cast<void*>(dv.grad) : kind == 3 ? static_cast<void*>(dv.m) : static_cast<void*>(dv.v);
                const void* s = kind == 0 ? hs.w : kind == 1 ? hs.scale : kind == 2 ? hs.grad : kind == 3 ? static_cast<const void*>(hs.m) : static_cast<const void*>(hs.v);
                const uint64_t b = kind == 0 ? p.wb : kind == 1 ? p.sb : kind == 2 ? p.gb : p.mb;
                add(h->copies_in[c], d, s, b);
                if (kind != 2) add(h->copies_out[c], d, s, b);      // the gradient is an input only
            }
        }
        ECO_CUDA_H(cudaEventCreateWithFlags(&h->ev_in[c], cudaEventDisableTiming));
        ECO_CUDA_H(cudaEventCreateWithFlags(&h->ev_run[c], cudaEventDisableTiming));
        ECO_CUDA_H(cudaEventCreateWithFlags(&h->ev_out[c], cudaEventDisableTiming));
    }
#undef ECO_CUDA_H
    *out = h;
    return ECO_OK;
}

eco_status eco_host_copies(const eco_host_ctx* h, uint64_t* h2d_copies, uint64_t* d2h_copies) {
    if (!h) return fail(nullptr, ECO_ERR_INVALID_ARG, "ctx is NULL");
    uint64_t in = 0, out = 0;
    for (const auto& v : h->copies_in) in += v.size();
    for (const auto& v : h->copies_out) out += v.size();
    if (h2d_copies) *h2d_copies = in;
    if (d2h_copies) *d2h_copies = out;
    return ECO_OK;
}

eco_status eco_host_step(eco_host_ctx* h, float lr, float beta1, float beta2, float eps, uint64_t step, uint64_t seed,
                         uint64_t* h2d_bytes, uint64_t* d2h_bytes) {
    if (!h) return fail(nullptr, ECO_ERR_INVALID_ARG, "ctx is NULL");
    if (eco_status st = check_hyper(nullptr, h->cfg, lr, beta1, beta2, eps, step)) return st;
    ECO_CUDA(nullptr, cudaSetDevice(h->device));
    uint64_t up = 0, down = 0;
    for (size_t c = 0; c < h->chunks.size(); ++c) {
        // the slot is free once the chunk that used it before has been copied out
        if (c >= static_cast<size_t>(h->n_slots)) ECO_CUDA(nullptr, cudaStreamWaitEvent(h->s_in, h->ev_out[c - h->n_slots], 0));
        for (const eco_host_ctx::Copy& cp : h->copies_in[c]) {
            ECO_CUDA(nullptr, cudaMemcpyAsync(cp.dev, cp.host, cp.bytes, cudaMemcpyHostToDevice, h->s_in));
            up += cp.bytes;
        }
        ECO_CUDA(nullptr, cudaEventRecord(h->ev_in[c], h->s_in));
        ECO_CUDA(nullptr, cudaStreamWaitEvent(h->s_run, h->ev_in[c], 0));
        eco_status rc = eco_step(h->ctxs[c], lr, beta1, beta2, eps, step, seed, h->s_run);
        if (rc != ECO_OK) { g_thread_error = h->ctxs[c]->err; cudaDeviceSynchronize(); return rc; }
        ECO_CUDA(nullptr, cudaEventRecord(h->ev_run[c], h->s_run));
        ECO_CUDA(nullptr, cudaStreamWaitEvent(h->s_out, h->ev_run[c], 0));
        for (const eco_host_ctx::Copy& cp : h->copies_out[c]) {
            ECO_CUDA(nullptr, cudaMemcpyAsync(cp.host, cp.dev, cp.bytes, cudaMemcpyDeviceToHost, h->s_out));
            down += cp.bytes;
        }
        ECO_CUDA(nullptr, cudaEventRecord(h->ev_out[c], h->s_out));
    }
    ECO_CUDA(nullptr, cudaStreamSynchronize(h->s_out));
    ECO_CUDA(nullptr, cudaStreamSynchronize(h->s_in));
    for (eco_ctx* c : h->ctxs) {
        eco_status rc = eco_check(c, h->s_run);
        if (rc != ECO_OK) { g_thread_error = c->err; return rc; }
    }
    if (h2d_bytes) *h2d_bytes = up;
    if (d2h_bytes) *d2h_bytes = down;
    return ECO_OK;
}

eco_status eco_dequantize(const eco_config* cfg, const void* w, const void* scale, int64_t rows, int64_t cols,
                          void* out, int out_bf16, int device, void* cuda_stream) {
    if (eco_status st = check_config(cfg, false)) return st;
    if (eco_status st = check_shape(*cfg, rows, cols, 0)) return st;
    ECO_CUDA(nullptr, cudaSetDevice(device));
    if (eco_status st = check_device_ptr(w, device, "w", 0, true)) return st;
    if (eco_status st = check_device_ptr(scale, device, "scale", 0, true)) return st;
    if (eco_status st = check_device_ptr(out, device, "out", 0, true)) return st;
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    const uint64_t quads = static_cast<uint64_t>(rows) * static_cast<uint64_t>((cols + 3) / 4);
    const uint32_t grid = static_cast<uint32_t>(std::max<uint64_t>(1, std::min<uint64_t>(static_cast<uint64_t>(sms) * 16, (quads + 255) / 256)));
    ECO_CUDA(nullptr, eco::launch_dequantize(launch_config(*cfg), static_cast<const uint8_t*>(w), scale, out,
                                             static_cast<uint64_t>(rows), static_cast<uint32_t>(cols), cfg->granularity,
                                             out_bf16 != 0, grid, static_cast<cudaStream_t>(cuda_stream)));
    return ECO_OK;
}

eco_status eco_step_host(const eco_config* cfg, const eco_tensor* tensors, size_t n, int device,
                         float lr, float beta1, float beta2, float eps, uint64_t step, uint64_t seed,
                         uint64_t* h2d_bytes, uint64_t* d2h_bytes) {
    if (eco_status st = check_config(cfg, true)) return st;
    if (eco_status st = check_hyper(nullptr, *cfg, lr, beta1, beta2, eps, step)) return st;
    eco_host_ctx* h = nullptr;
    if (eco_status st = eco_host_create(&h, cfg, tensors, n, device)) return st;
    const eco_status st = eco_host_step(h, lr, beta1, beta2, eps, step, seed, h2d_bytes, d2h_bytes);
    eco_host_destroy(h);
    return st;
}

// ---------------------------------------------------------------------------
// eco_step_static: the per-tensor-scale step with every byte of library-side
// device memory taken from one fixed array that is part of the loaded module.
// ---------------------------------------------------------------------------
}  // extern "C"

namespace {

constexpr uint32_t kStaticMaxTensors = ECO_STATIC_MAX_TENSORS;
constexpr uint32_t kStaticMaxUnits = 32768;   // work units of 4096 parameters: 2^27 parameters per call
static_assert(sizeof(TensorDesc) % 8 == 0, "tables are laid out back to back");

// Layout of the array: descriptors, amax slots of this step, amax slots the second kernel clears,
// saved old scales, unit -> tensor table.
struct StaticScratch {
    TensorDesc descs[kStaticMaxTensors];
    uint32_t amax[kStaticMaxTensors];
    uint32_t amax_next[kStaticMaxTensors];
    float s_old[kStaticMaxTensors];
    uint32_t unit_tensor[kStaticMaxUnits];
};

// Lives in every GPU that loads the library, from load to exit (about 135 KB).  In host code this name
// is only a handle: the device address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
StaticScratch* g_static_ptr[kMaxDevices] = {};

// Device address of the array on `device` (which must be current); resolved once per device.
eco_status static_scratch_address(int device, StaticScratch** out) {
    if (device < 0 || device >= kMaxDevices) return fail(nullptr, ECO_ERR_INVALID_ARG, "device ordinal %d out of range", device);
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p)
            return fail(nullptr, ECO_ERR_CUDA, "cudaGetSymbolAddress(static scratch) on device %d failed: %s", device,
                        cudaGetErrorString(e));
        g_static_ptr[device] = static_cast<StaticScratch*>(p);
    }
    *out = g_static_ptr[device];
    return ECO_OK;
}

}  // namespace

extern "C" {

eco_status eco_step_static(const eco_config* cfg, const eco_tensor* tensors, size_t n, int device,
                           float lr, float beta1, float beta2, float eps, uint64_t step, uint64_t seed,
                           void* cuda_stream) {
    if (eco_status st = check_config(cfg, true)) return st;
    if (cfg->granularity != ECO_SCALE_PER_TENSOR)
        return fail(nullptr, ECO_ERR_UNSUPPORTED, "eco_step_static handles ECO_SCALE_PER_TENSOR only");
    if (cfg->injection == ECO_INJECT_EXACT)
        return fail(nullptr, ECO_ERR_UNSUPPORTED, "eco_step_static has no error buffers: ECO_INJECT_EXACT is not available");
    if (!tensors || n == 0) return fail(nullptr, ECO_ERR_INVALID_ARG, "empty tensor list");
    if (n > kStaticMaxTensors)
        return fail(nullptr, ECO_ERR_INVALID_ARG, "eco_step_static takes at most %u tensors per call (got %zu)",
                    kStaticMaxTensors, n);
    if (eco_status st = check_hyper(nullptr, *cfg, lr, beta1, beta2, eps, step)) return st;
    const bool adam = cfg->optimizer == ECO_OPT_ADAM;
    const uint64_t rpu = static_cast<uint64_t>(eco::rows_per_unit());
    static thread_local StaticScratch host;          // host image of the tables (no heap use either)
    uint64_t units = 0, total = 0;
    for (size_t i = 0; i < n; ++i) {
        const eco_tensor& t = tensors[i];
        if (eco_status st = check_shape(*cfg, t.rows, t.cols, i)) return st;
        if ((static_cast<uint64_t>(t.row_offset) * static_cast<uint64_t>(t.cols)) % 4 != 0)
            return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: row_offset * cols must be a multiple of 4", i);
        if (static_cast<unsigned __int128>(static_cast<uint64_t>(t.row_offset) + static_cast<uint64_t>(t.rows)) *
                static_cast<unsigned __int128>(t.cols) >= (static_cast<unsigned __int128>(1) << 34))
            return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: (row_offset + rows) * cols must be < 2^34", i);
        if (adam != (t.v != nullptr)) return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: v must be given for Adam and NULL for SGDM", i);
        for (size_t j = 0; j < i; ++j)
            if (tensors[j].tensor_id == t.tensor_id) return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: duplicate tensor_id %u", i, t.tensor_id);
        const void* bufs[5] = {t.w, t.scale, t.grad, t.m, t.v};
        const char* names[5] = {"w", "scale", "grad", "m", "v"};
        for (int b = 0; b < (adam ? 5 : 4); ++b) {
            if (!bufs[b]) return fail(nullptr, ECO_ERR_INVALID_ARG, "tensor %zu: %s is NULL", i, names[b]);
            if (reinterpret_cast<uintptr_t>(bufs[b]) & 15) return fail(nullptr, ECO_ERR_ALIGNMENT, "tensor %zu: %s is not 16-byte aligned", i, names[b]);
        }
        TensorDesc d;
        std::memset(&d, 0, sizeof d);
        d.w = static_cast<uint8_t*>(t.w);
        d.scale = t.scale;
        d.grad = static_cast<const uint16_t*>(t.grad);
        d.m = t.m;
        d.v = t.v;
        d.numel = static_cast<uint64_t>(t.rows) * static_cast<uint64_t>(t.cols);
        d.cols = static_cast<uint32_t>(t.cols);
        d.blocks_per_row = static_cast<uint32_t>((t.cols + 127) / 128);
        d.n_blocks = (d.numel + 127) / 128;
        d.tensor_id = t.tensor_id;
        d.slot = static_cast<uint32_t>(i);
        d.index_base = static_cast<uint64_t>(t.row_offset) * static_cast<uint64_t>(t.cols);
        const uint64_t nu = (d.n_blocks + rpu - 1) / rpu;
        total += d.numel;
        if (units + nu > kStaticMaxUnits)
            return fail(nullptr, ECO_ERR_INVALID_ARG,
                        "eco_step_static takes at most %llu parameters per call (%u units of %llu); the list has more",
                        static_cast<unsigned long long>(kStaticMaxUnits * rpu * 128), kStaticMaxUnits,
                        static_cast<unsigned long long>(rpu * 128));
        d.first_unit = static_cast<uint32_t>(units);
        host.descs[i] = d;
        for (uint64_t u = 0; u < nu; ++u) host.unit_tensor[units + u] = static_cast<uint32_t>(i);
        units += nu;
    }
    (void)total;
    ECO_CUDA(nullptr, cudaSetDevice(device));
    StaticScratch* dev = nullptr;
    if (eco_status st = static_scratch_address(device, &dev)) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // The array keeps whatever the previous call left: upload this call's tables and zero both amax ranges.
    ECO_CUDA(nullptr, cudaMemcpyAsync(dev->descs, host.descs, n * sizeof(TensorDesc), cudaMemcpyHostToDevice, stream));
    ECO_CUDA(nullptr, cudaMemcpyAsync(dev->unit_tensor, host.unit_tensor, units * sizeof(uint32_t), cudaMemcpyHostToDevice, stream));
    ECO_CUDA(nullptr, cudaMemsetAsync(dev->amax, 0, 2 * kStaticMaxTensors * sizeof(uint32_t), stream));
    const LaunchConfig lc = launch_config(*cfg);
    const StepParams P = derive_params(*cfg, lr, beta1, beta2, eps, step, seed);
    ECO_CUDA(nullptr, eco::launch_tensor_amax(lc, dev->descs, dev->unit_tensor, static_cast<uint32_t>(units), P, dev->amax,
                                              dev->s_old, stream));
    ECO_CUDA(nullptr, eco::launch_tensor_apply(lc, dev->descs, dev->unit_tensor, static_cast<uint32_t>(units), P, dev->amax,
                                               dev->amax_next, dev->s_old, false, stream));
    // the host image is reused by the next call on this thread: wait until the copies have read it
    ECO_CUDA(nullptr, cudaStreamSynchronize(stream));
    return ECO_OK;
}

}  // extern "C"
