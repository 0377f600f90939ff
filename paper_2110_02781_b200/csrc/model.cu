// Model object and the C ABI around it: validation, memory layout inside the caller's workspace,
// stage forward / backward / SGD, re-homing of weights after a new partition, snapshots, the
// per-unit profile and the kernel trace.
#include <algorithm>
#include <cstdlib>
#include <string>
#include <cstring>
#include <new>
#include <type_traits>
#include "model.h"

using namespace ftp;

namespace {

static long long g_launches = 0;

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Every buffer carved out of the workspace is followed by a 256-byte guard zone filled with a pattern when the model is
// built; ftp_check_guards finds a kernel that wrote past the end of its buffer (the stand-in for a memory checker).
constexpr size_t kGuardBytes = 256;
constexpr unsigned char kGuardByte = 0xA5;
struct Bump {
    char* base;
    size_t off;
    std::vector<size_t>* guards;          // offsets of the guard zones (nullable)
    void* take(size_t bytes) {
        off = align_up(off, 256);
        void* p = base ? base + off : reinterpret_cast<void*>(off + 256);   // dry run: fake, never dereferenced
        off += bytes;
        off = align_up(off, 256);
        if (guards) guards->push_back(off);
        off += kGuardBytes;
        return p;
    }
};

const char* kKernelNames[K_COUNT] = {
    "conv_fwd_f32", "conv_dgrad_f32", "conv_wgrad_f32", "bn_stats", "bn_finalize", "bn_apply", "bn_bwd_reduce",
    "bn_bwd_finalize", "bn_bwd_apply", "act_bias_bwd", "dw_fwd", "dw_dgrad", "dw_wgrad", "maxpool_fwd", "maxpool_bwd",
    "gap_fwd", "gap_bwd", "softmax_ce", "sgd", "act_fwd", "act_bwd", "copy", "tc_gemm_bf16_fwd", "tc_gemm_bf16_dgrad",
    "tc_gemm_bf16_wgrad", "conv_fwd_bf16_simt", "conv_dgrad_bf16_simt", "conv_wgrad_bf16_simt",
    "tc_gemm_tf32x3_fwd", "tc_gemm_tf32x3_dgrad", "tc_gemm_tf32x3_wgrad"};

// Brackets one launcher call with events when tracing is on.
struct Scope {
    ftp_model* m;
    cudaStream_t st;
    TraceSlot* slot;
    Scope(ftp_model* m_, cudaStream_t st_, int kernel, int unit, int op, int bwd, double bytes, double flops, int nk = 1)
        : m(m_), st(st_), slot(nullptr) {
        g_launches += nk;
        if (!m->trace) return;
        if (m->tr_used == m->tr.size()) {
            TraceSlot s{};
            if (cudaEventCreate(&s.e0) != cudaSuccess || cudaEventCreate(&s.e1) != cudaSuccess) return;
            m->tr.push_back(s);
        }
        slot = &m->tr[m->tr_used++];
        slot->rec = ftp_trace_rec{kernel, unit, op, bwd, 0.f, bytes, flops};
        cudaEventRecord(slot->e0, st);
    }
    ~Scope() { if (slot) cudaEventRecord(slot->e1, st); }
};

bool is_contraction(int kind) { return kind == FTP_CONV1D || kind == FTP_CONV2D || kind == FTP_FC; }
bool is_pointwise_op(const Op& o);
bool is_3x3_op(const Op& o);

// ---- shapes, parameter offsets, validation ------------------------------------------------------
ftp_status plan_ops(const ftp_layer_desc* layers, int n, const ftp_model_cfg* cfg, ftp_model& m) {
    FTP_REQUIRE(layers && cfg, FTP_EINVAL, "build_model: null argument");
    FTP_REQUIRE(n >= 1, FTP_EINVAL, "build_model: empty layer list");
    FTP_REQUIRE(cfg->batch >= 1 && cfg->in_c >= 1 && cfg->in_h >= 1 && cfg->in_w >= 1 && cfg->n_classes >= 1, FTP_EINVAL,
                "build_model: batch, input shape and class count must be positive");
    FTP_REQUIRE(cfg->precision == FTP_FP32 || cfg->precision == FTP_BF16, FTP_EINVAL, "build_model: unknown precision %d", cfg->precision);
    FTP_REQUIRE(cfg->max_stages >= 1 && cfg->max_stages <= 64, FTP_EINVAL, "build_model: max_stages must be in 1..64");
    FTP_REQUIRE(layers[0].unit == 0, FTP_EINVAL, "build_model: the first op must belong to unit 0");
    FTP_REQUIRE(layers[n - 1].kind == FTP_SOFTMAX_CE, FTP_EINVAL, "build_model: the last op must be SOFTMAX_CE");
    m.cfg = *cfg;
    m.esize = cfg->precision == FTP_BF16 ? 2 : 4;
    m.ops.assign(n, Op{});
    int H = cfg->in_h, W = cfg->in_w, C = cfg->in_c;
    const int N = cfg->batch;
    long long poff = 0, soff = 0;
    m.unit_first.clear(); m.unit_last.clear();
    for (int i = 0; i < n; ++i) {
        const ftp_layer_desc& d = layers[i];
        Op& o = m.ops[i];
        o.d = d;
        FTP_REQUIRE(i == 0 || d.unit == layers[i - 1].unit || d.unit == layers[i - 1].unit + 1, FTP_EINVAL,
                    "build_model: op %d: unit ids must be non-decreasing without gaps", i);
        if (i == 0 || d.unit != layers[i - 1].unit) { m.unit_first.push_back(i); m.unit_last.push_back(i); }
        else m.unit_last.back() = i;
        o.N = N; o.H = H; o.W = W; o.C = C;
        o.w_off = o.b_off = o.rm_off = o.rv_off = -1;
        o.w_cnt = o.b_cnt = 0;
        o.gslot = -1; o.galias = i; o.addend_of = -1;
        o.Ho = H; o.Wo = W; o.Co = C;
        FTP_REQUIRE(d.act >= 0 && d.act <= 2, FTP_EINVAL, "build_model: op %d: unknown activation %d", i, d.act);
        switch (d.kind) {
            case FTP_CONV1D: case FTP_CONV2D: case FTP_FC: {
                FTP_REQUIRE(d.cin == C && d.cout >= 1, FTP_EINVAL, "build_model: op %d: cin %d does not match the incoming %d channels", i, d.cin, C);
                int kh = 1, kw = 1, st = 1, ph = 0, pw = 0;
                if (d.kind == FTP_CONV1D) { FTP_REQUIRE(H == 1, FTP_EINVAL, "build_model: op %d: CONV1D needs H == 1", i); kw = d.k; st = d.stride; pw = d.pad; }
                else if (d.kind == FTP_CONV2D) { kh = kw = d.k; st = d.stride; ph = pw = d.pad; }
                else FTP_REQUIRE(H == 1 && W == 1, FTP_EINVAL, "build_model: op %d: FC needs a 1x1 input (pool first)", i);
                FTP_REQUIRE(kw >= 1 && st >= 1 && pw >= 0, FTP_EINVAL, "build_model: op %d: bad kernel geometry", i);
                o.Ho = (H + 2 * ph - kh) / st + 1; o.Wo = (W + 2 * pw - kw) / st + 1; o.Co = d.cout;
                FTP_REQUIRE(H + 2 * ph >= kh && W + 2 * pw >= kw, FTP_EINVAL, "build_model: op %d: kernel larger than the padded input", i);
                o.g = ConvGeom{N, H, W, C, o.Ho, o.Wo, o.Co, kh, kw, st, ph, pw};
                o.w_off = poff; o.w_cnt = (long long)kh * kw * C * d.cout; poff += o.w_cnt;
                if (d.has_bias) { o.b_off = poff; o.b_cnt = d.cout; poff += o.b_cnt; }
                break;
            }
            case FTP_DWCONV3x3:
                FTP_REQUIRE(d.cin == C && d.cout == C && d.k == 3 && d.pad == 1 && d.stride >= 1, FTP_EINVAL,
                            "build_model: op %d: depthwise needs cin == cout == incoming channels, k 3, pad 1", i);
                o.Ho = (H + 2 - 3) / d.stride + 1; o.Wo = (W + 2 - 3) / d.stride + 1;
                o.g = ConvGeom{N, H, W, C, o.Ho, o.Wo, C, 3, 3, d.stride, 1, 1};
                o.w_off = poff; o.w_cnt = 9LL * C; poff += o.w_cnt;
                break;
            case FTP_BN:
                FTP_REQUIRE(d.cin == C, FTP_EINVAL, "build_model: op %d: BN over %d channels but %d arrive", i, d.cin, C);
                o.w_off = poff; o.w_cnt = C; poff += C;
                o.b_off = poff; o.b_cnt = C; poff += C;
                o.rm_off = soff; soff += C; o.rv_off = soff; soff += C;
                break;
            case FTP_ACT: break;
            case FTP_ADD_RESIDUAL: {
                const int s = d.residual_src;
                FTP_REQUIRE(s >= -1 && s < i - 1, FTP_EINVAL, "build_model: op %d: residual_src %d out of range", i, s);
                FTP_REQUIRE(s >= m.unit_first.back() - 1, FTP_EINVAL, "build_model: op %d: a residual connection may not cross a unit edge", i);
                const int sh = s < 0 ? cfg->in_h : m.ops[s].Ho, sw = s < 0 ? cfg->in_w : m.ops[s].Wo, sc = s < 0 ? cfg->in_c : m.ops[s].Co;
                FTP_REQUIRE(sh == H && sw == W && sc == C, FTP_EINVAL, "build_model: op %d: residual shapes differ", i);
                FTP_REQUIRE(i >= 1 && layers[i - 1].kind == FTP_BN && layers[i - 1].act == FTP_ACT_NONE && layers[i - 1].unit == d.unit,
                            FTP_EUNSUPPORTED, "build_model: op %d: a residual add must follow a BN without activation", i);
                break;
            }
            case FTP_MAXPOOL2:
                FTP_REQUIRE(H >= 2 && W >= 2, FTP_EINVAL, "build_model: op %d: max-pool input smaller than 2x2", i);
                o.Ho = H / 2; o.Wo = W / 2;
                break;
            case FTP_GAP: o.Ho = 1; o.Wo = 1; break;
            case FTP_SOFTMAX_CE:
                FTP_REQUIRE(i == n - 1, FTP_EINVAL, "build_model: op %d: SOFTMAX_CE must be the last op", i);
                FTP_REQUIRE(H == 1 && W == 1 && C == cfg->n_classes, FTP_EINVAL, "build_model: the loss expects %d logits, got %dx%dx%d", cfg->n_classes, H, W, C);
                FTP_REQUIRE(i >= 1 && layers[i - 1].kind == FTP_FC && layers[i - 1].act == FTP_ACT_NONE && layers[i - 1].unit == d.unit,
                            FTP_EUNSUPPORTED, "build_model: SOFTMAX_CE must directly follow an FC op of the same unit");
                o.Ho = o.Wo = o.Co = 1;
                break;
            default: return fail(FTP_EINVAL, "build_model: op %d: unknown kind %d", i, d.kind);
        }
        o.in_elems = (long long)N * H * W * C;
        o.out_elems = d.kind == FTP_SOFTMAX_CE ? 1 : (long long)N * o.Ho * o.Wo * o.Co;
        FTP_REQUIRE(o.in_elems < (1LL << 31) && o.out_elems < (1LL << 31), FTP_ERANGE, "build_model: op %d: tensor too large", i);
        o.out_f32 = d.kind == FTP_SOFTMAX_CE || (d.kind == FTP_FC && i + 1 < n && layers[i + 1].kind == FTP_SOFTMAX_CE);
        H = o.Ho; W = o.Wo; C = o.Co;
    }
    m.L = (int)m.unit_first.size();
    m.P = poff; m.R = soff;
    m.unit_p_off.assign(m.L, 0); m.unit_p_cnt.assign(m.L, 0); m.unit_s_off.assign(m.L, 0); m.unit_s_cnt.assign(m.L, 0);
    for (int u = 0; u < m.L; ++u) {
        long long p0 = -1, p1 = 0, s0 = -1, s1 = 0;
        for (int i = m.unit_first[u]; i <= m.unit_last[u]; ++i) {
            const Op& o = m.ops[i];
            if (o.w_off >= 0) { if (p0 < 0) p0 = o.w_off; p1 = o.w_off + o.w_cnt; }
            if (o.b_off >= 0) p1 = o.b_off + o.b_cnt;
            if (o.rm_off >= 0) { if (s0 < 0) s0 = o.rm_off; s1 = o.rv_off + o.C; }
        }
        m.unit_p_off[u] = p0 < 0 ? (u ? m.unit_p_off[u - 1] + m.unit_p_cnt[u - 1] : 0) : p0;
        m.unit_p_cnt[u] = p0 < 0 ? 0 : p1 - p0;
        m.unit_s_off[u] = s0 < 0 ? (u ? m.unit_s_off[u - 1] + m.unit_s_cnt[u - 1] : 0) : s0;
        m.unit_s_cnt[u] = s0 < 0 ? 0 : s1 - s0;
    }
    // fuse "BN (no activation) -> residual add"
    for (int i = 0; i + 1 < n; ++i)
        if (m.ops[i + 1].d.kind == FTP_ADD_RESIDUAL) { m.ops[i].fused_add = true; m.ops[i + 1].skip = true; }
    // A batch norm inside a unit whose only reader can normalise while it loads (a depthwise convolution, or a 1x1
    // convolution on the split-tf32 tensor-core kernel) is never applied in memory: only its statistics and
    // per-channel constants are computed, and forward and weight gradient of the reader work from the BN's input.
    // FTP_FUSE_BN (A/B measurements): bit 0 = into depthwise readers, bit 1 = into 1x1 readers, bit 2 = into stride-2
    // depthwise readers only, 0 = every batch norm stores its output.  Default: bits 0 and 1 in float models; bit 2 in
    // bf16 models, whose stride-1 depthwise kernels are bound by instruction issue and lose more to the extra arithmetic
    // per loaded element than the saved pass gives back.
    const char* fe = std::getenv("FTP_FUSE_BN");
    const int fuse = fe ? std::atoi(fe) : (cfg->precision == FTP_FP32 ? 3 : 4);
    const char* fm = std::getenv("FTP_FUSE_MAX_MB");                  // only batch norms whose output is at most this large (A/B measurements)
    const double fuse_max_bytes = fm ? std::atof(fm) * 1e6 : 1e30;
    for (int i = 0; fuse && i + 1 < n; ++i) {
        Op& o = m.ops[i];
        const Op& c = m.ops[i + 1];
        if (o.d.kind != FTP_BN || o.fused_add || c.d.unit != o.d.unit) continue;
        bool other_reader = false;
        for (int j = i + 2; j < n; ++j) other_reader |= m.ops[j].d.kind == FTP_ADD_RESIDUAL && m.ops[j].d.residual_src == i;
        if (other_reader || (double)o.out_elems * m.esize > fuse_max_bytes) continue;
        void* const al = reinterpret_cast<void*>(256);
        if (c.d.kind == FTP_DWCONV3x3) o.defer = (fuse & 1) != 0 || ((fuse & 4) != 0 && c.g.stride == 2);
        else if ((fuse & 2) && cfg->precision == FTP_FP32 && is_pointwise_op(c) && tc32_supported(c.N * c.Ho * c.Wo, c.Co, c.C, al, al, al, nullptr)) o.defer = true;
    }
    return FTP_OK;
}

// ---- gradient-buffer plan: which slot holds the gradient of each op's output ------------------------
ftp_status plan_gradients(ftp_model& m, int* n_slots) {
    const int n = (int)m.ops.size();
    std::vector<int> refc;               // per slot: readers still to come
    std::vector<int> freel;
    std::vector<int> pending(n + 1, -1); // pending[j+1]: op whose output-gradient buffer must be added into grad(out[j])
    // A freed slot is handed out again as late as possible (oldest first, and only once `spare` slots exist): the weight
    // gradient that reads a gradient buffer runs on the second stream, and the main stream has to wait for it before the
    // buffer is overwritten.  FTP_GRAD_SLOTS: the number of slots before any is reused (A/B measurements; at least the
    // liveness minimum is always allocated).
    const char* gs = std::getenv("FTP_GRAD_SLOTS");
    const int spare = gs ? std::atoi(gs) : 48;      // measured: 16 -> 48 slots 3.280 -> 3.255 ms (MobileNetV2 32x32 float), 5.03 -> 4.97 ms (224x224 bf16); no gain beyond
    auto alloc = [&]() {
        if (!freel.empty() && (int)refc.size() >= spare) { int s = freel.front(); freel.erase(freel.begin()); refc[s] = 1; return s; }
        refc.push_back(1);
        return (int)refc.size() - 1;
    };
    auto release = [&](int s) { if (s >= 0 && --refc[s] == 0) freel.push_back(s); };
    for (int i = n - 1; i >= 0; --i) {
        Op& o = m.ops[i];
        if (o.d.kind == FTP_SOFTMAX_CE) { m.ops[i - 1].gslot = -2; continue; }
        const int k = o.galias;                         // buffer this op reads its output gradient from
        const int s = m.ops[k].gslot;
        FTP_REQUIRE(s != -1, FTP_ESTATE, "build_model: op %d has no consumer for its output", i);
        if (o.d.kind == FTP_ADD_RESIDUAL) {
            m.ops[i - 1].galias = k; m.ops[i - 1].gslot = s;
            const int src = o.d.residual_src;
            FTP_REQUIRE(pending[src + 1] < 0, FTP_EUNSUPPORTED, "build_model: op %d: two residual adds share one source", i);
            pending[src + 1] = k;
            if (s >= 0) refc[s] += 1;                   // readers: op i-1 (already counted as op i's read) and the addend user
            continue;
        }
        if (i > 0) {
            m.ops[i - 1].gslot = alloc();
            if (pending[i] >= 0) o.addend_of = pending[i];
        }
        // after op i has run: its own output gradient is consumed, and so is the addend it folded in
        if (s >= 0) release(s);
        if (o.addend_of >= 0) release(m.ops[o.addend_of].gslot);
    }
    *n_slots = (int)refc.size();
    return FTP_OK;
}

// ---- memory layout inside the workspace --------------------------------------------------------------
ftp_status layout(ftp_model& m, char* dev_base, size_t* dev_total, size_t* pinned_total) {
    m.guards.clear();
    Bump bp{dev_base, 0, &m.guards};
    const int n = (int)m.ops.size();
    const size_t es = (size_t)m.esize;
    m.arena.assign(m.cfg.max_stages, Arena{});
    for (auto& a : m.arena) {
        a.w = (float*)bp.take((size_t)m.P * 4);
        a.m = (float*)bp.take((size_t)m.P * 4);
        a.run = (float*)bp.take((size_t)std::max<long long>(m.R, 1) * 4);
        a.wb = m.cfg.precision == FTP_BF16 ? (__nv_bfloat16*)bp.take((size_t)m.P * 2) : nullptr;
        a.wbt = m.cfg.precision == FTP_BF16 ? (__nv_bfloat16*)bp.take((size_t)m.P * 2) : nullptr;
        const bool f32 = m.cfg.precision == FTP_FP32;
        a.wl = f32 ? (float*)bp.take((size_t)m.P * 4) : nullptr;
        a.wt = f32 ? (float*)bp.take((size_t)m.P * 4) : nullptr;
        a.wtl = f32 ? (float*)bp.take((size_t)m.P * 4) : nullptr;
    }
    {   // table of the 1x1-convolution matrices for the batched transposition
        m.tp_host.clear(); m.tp_first.assign(m.L + 1, 0);
        int tile0 = 0, u_next = 0;
        for (int i = 0; i < n; ++i) {
            const Op& o = m.ops[i];
            while (u_next <= o.d.unit) m.tp_first[u_next++] = (int)m.tp_host.size();
            if (m.cfg.precision == FTP_FP32 && is_pointwise_op(o) && o.d.kind != FTP_FC) {
                m.tp_host.push_back(TransposeEntryDev{o.w_off, o.C, o.Co, tile0, 1});
                tile0 += ((o.C + 31) / 32) * ((o.Co + 31) / 32);
            } else if (m.cfg.precision == FTP_BF16 && (is_pointwise_op(o) || is_3x3_op(o))) {
                const int taps = o.g.kh * o.g.kw;
                m.tp_host.push_back(TransposeEntryDev{o.w_off, o.C, o.Co, tile0, taps});
                tile0 += taps * ((o.C + 31) / 32) * ((o.Co + 31) / 32);
            }
        }
        while (u_next <= m.L) m.tp_first[u_next++] = (int)m.tp_host.size();
        m.tp_host.push_back(TransposeEntryDev{0, 0, 0, tile0, 1});
        m.tp_dev = (TransposeEntryDev*)bp.take(m.tp_host.size() * sizeof(TransposeEntryDev));
    }
    m.grad = (float*)bp.take((size_t)m.P * 4);
    m.state_backup = (float*)bp.take((size_t)std::max<long long>(m.R, 1) * 4);
    size_t max_act = 0, red = 0, dwp = 0, foldd = 0, dpre = 0, finp = 64, finc = 1, fcin = 64;
    for (int i = 0; i < n; ++i) {
        Op& o = m.ops[i];
        const size_t obytes = (size_t)o.out_elems * (o.out_f32 ? 4 : es);
        o.out = (o.fused_add || o.defer) ? nullptr : bp.take(obytes);  // a fused BN writes into the add's buffer, a deferred one nowhere
        if (!o.out_f32 && i + 1 < n) max_act = std::max(max_act, obytes);
        const long long Mout = (long long)o.N * o.Ho * o.Wo;
        if (o.d.kind == FTP_BN) {
            const size_t stride = align_up((size_t)o.C * 4, 256) / 4;
            float* t = (float*)bp.take((6 * stride + 5 * (size_t)o.C) * 4);
            o.scale = t; o.shift = t + stride; o.mean = t + 2 * stride; o.mean_lo = t + 3 * stride; o.rstd = t + 4 * stride; o.offset = t + 5 * stride;
            o.coef = t + 6 * stride;
            o.fold = make_fold(Mout, o.C, m.esize);
            foldd = std::max(foldd, std::max(fold_partial_doubles(o.fold), producer_partial_doubles(Mout, o.C)));
            finp = std::max(finp, fin_part_doubles(o.C, 1)); finc = std::max(finc, fin_counter_count(o.C, 1));
        } else if (is_contraction(o.d.kind)) {
            finp = std::max(finp, fin_part_doubles(o.Co, 1)); finc = std::max(finc, fin_counter_count(o.Co, 1));
            red = std::max(red, std::max(conv_wgrad_scratch_floats(o.g), conv_gemm_scratch_floats(o.g)));
            if (o.d.act == FTP_ACT_NONE && o.b_off < 0) red = std::max(red, stem_wgrad_scratch_floats(o.g));
            red = std::max(red, tc32_wgrad_scratch_floats(Mout, o.C, o.Co));
            red = std::max(red, std::max(tc32_gemm_scratch_floats((int)Mout, o.Co, o.C), tc32_gemm_scratch_floats((int)Mout, o.C, o.Co)));
            if (m.cfg.precision == FTP_BF16) {
                red = std::max(red, std::max(tc_wgrad_scratch_floats(Mout, o.C, o.Co), tc_wgrad3x3_scratch_floats(Mout, o.C, o.Co)));
                const int kk = o.g.kh * o.g.kw;
                red = std::max(red, std::max(tc_gemm_scratch_floats((int)Mout, o.Co, kk * o.C), tc_gemm_scratch_floats((int)Mout, o.C, kk * o.Co)));
            }
            o.fold = make_fold(Mout, o.Co, o.out_f32 ? 4 : m.esize);
            if (o.d.act != FTP_ACT_NONE || o.d.has_bias) foldd = std::max(foldd, fold_partial_doubles(o.fold));
            if (o.d.act != FTP_ACT_NONE) dpre = std::max(dpre, obytes);
            if (o.d.kind == FTP_FC) fcin = std::max(fcin, (size_t)o.in_elems);
        } else if (o.d.kind == FTP_DWCONV3x3) {
            red = std::max(red, dwconv_wgrad_scratch_floats(o.g));
            dwp = std::max(dwp, dwconv_wgrad_scratch_floats(o.g));
            foldd = std::max(foldd, dwconv_bwd_stats_doubles(o.g));
            finp = std::max(finp, fin_part_doubles(o.C, 9)); finc = std::max(finc, fin_counter_count(o.C, 9));
        }
    }
    int n_slots = 0;
    ftp_status s = plan_gradients(m, &n_slots);
    if (s != FTP_OK) return s;
    m.slot_bytes = align_up(std::max<size_t>(max_act, 256), 256);
    m.slots.assign(n_slots, nullptr);
    for (auto& p : m.slots) p = bp.take(m.slot_bytes);
    m.red_floats = std::max<size_t>(red, 64); m.red_scratch = (float*)bp.take(m.red_floats * 4);
    m.red_side = (float*)bp.take(m.red_floats * 4);
    for (int k = 0; k < 4; ++k) m.dw_part[k] = (float*)bp.take(std::max<size_t>(dwp, 64) * 4);
    m.fold_doubles = std::max<size_t>(foldd, 64); m.fold_scratch = (double*)bp.take(m.fold_doubles * 8);
    m.dpre_bytes = std::max<size_t>(dpre, 256); m.dpre = bp.take(m.dpre_bytes);
    m.tc_err = (int*)bp.take(256);
    m.fc_in = (float*)bp.take(fcin * 4); m.fc_din = (float*)bp.take(fcin * 4);
    m.fin.part = (double*)bp.take(finp * 8);
    m.fin_counter_bytes = finc * 4; m.fin.counters = (unsigned*)bp.take(m.fin_counter_bytes);
    m.fin_side.part = (double*)bp.take(finp * 8); m.fin_side.counters = (unsigned*)bp.take(m.fin_counter_bytes);
    m.dlogits = (float*)bp.take((size_t)m.cfg.batch * m.cfg.n_classes * 4);
    m.per_sample = (float*)bp.take((size_t)m.cfg.batch * 4);
    m.loss_dev = (float*)bp.take(256);
    m.labels_dev = (int32_t*)bp.take((size_t)m.cfg.batch * 4);
    m.input_dev = bp.take((size_t)m.cfg.batch * m.cfg.in_h * m.cfg.in_w * m.cfg.in_c * es);
    *dev_total = align_up(bp.off, 256);
    *pinned_total = 256;
    return FTP_OK;
}

#define CUDA_OK(call)                                                                      \
    do {                                                                                   \
        cudaError_t e_ = (call);                                                           \
        if (e_ != cudaSuccess) return fail(FTP_ECUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
    } while (0)

bool is_pointwise_op(const Op& o) {
    return o.d.kind == FTP_CONV2D && o.g.kh == 1 && o.g.kw == 1 && o.g.stride == 1 && o.g.ph == 0 && o.d.act == FTP_ACT_NONE && o.b_off < 0;
}

bool is_3x3_op(const Op& o) {
    return o.d.kind == FTP_CONV2D && o.g.kh == 3 && o.g.kw == 3 && o.g.stride == 1 && o.g.ph == 1 && o.g.pw == 1 && o.d.act == FTP_ACT_NONE && o.b_off < 0;
}

// Rebuild the transposed copies of the convolution matrices of units [a, b) from the float masters: one batched launch
// per owning arena (float models: the 1x1 matrices with their lo parts; bf16 models: the 1x1 and 3x3 matrices).
void refresh_transposed(ftp_model* m, int a, int b, cudaStream_t st) {
    for (int u = a; u < b;) {
        int v = u + 1;
        while (v < b && m->owner[v] == m->owner[u]) ++v;
        const Arena& ar = m->arena[m->owner[u]];
        const int e0 = m->tp_first[u], e1 = m->tp_first[v];
        if (e1 > e0) {
            const int tiles = m->tp_host[e1].tile0 - m->tp_host[e0].tile0;
            if (m->cfg.precision == FTP_FP32) transpose_split_f32(m->tp_dev + e0, e1 - e0, m->tp_host[e0].tile0, tiles, ar.w, ar.wt, ar.wtl, st);
            else if (ar.wbt) transpose_bf16_batched(m->tp_dev + e0, e1 - e0, m->tp_host[e0].tile0, tiles, ar.w, ar.wbt, st);
        }
        u = v;
    }
}

ftp_status check_launches(const char* where) {
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(FTP_ECUDA, "%s: %s", where, cudaGetErrorString(e));
    return FTP_OK;
}

inline bool a16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }


// ---- forward of a unit range ------------------------------------------------------------------------------
template <typename T>
ftp_status fwd_range(ftp_model* m, int a, int b, const void* act_in, void* act_out, const int32_t* labels, float* loss_out,
                     cudaStream_t st) {
    const int first = m->unit_first[a], last = m->unit_last[b - 1];
    const double es = (double)m->esize;
    PartialSums next_ps{nullptr, 0, 1};
    m->stage_in[first] = act_in;
    for (int i = first; i <= last; ++i) {
        Op& o = m->ops[i];
        const int u = o.d.unit;
        if (m->unit_events && i == m->unit_first[u]) cudaEventRecord(m->ev_f[u], st);
        const void* in = (i == first) ? act_in : m->cur_out[i - 1];
        void* out = (i == last && act_out) ? act_out : o.out;
        if (o.fused_add) out = (i + 1 == last && act_out) ? act_out : m->ops[i + 1].out;
        const Arena& ar = m->arena[m->owner[u]];
        const long long Mout = (long long)o.N * o.Ho * o.Wo;
        // a producer whose output goes straight into a batch norm of this range leaves the statistics as it stores
        PartialSums have_ps = next_ps;
        next_ps.entries = 0;
        ColStatsReq req{m->fold_scratch, nullptr, &next_ps};
        const ColStatsReq* stats_req = nullptr;
        if (m->producer_stats && i + 1 <= last && m->ops[i + 1].d.kind == FTP_BN && o.d.kind != FTP_BN) { req.fold = &m->ops[i + 1].fold; stats_req = &req; }
        // the input is what a deferred batch norm read: this op normalises as it loads
        BnXform xfv{nullptr, nullptr, nullptr, 0.f, 0.f};
        const BnXform* xf = nullptr;
        if (i > first && m->ops[i - 1].defer) { const Op& bn = m->ops[i - 1]; xfv = make_xform(bn.mean, bn.scale, bn.offset, bn.d.act); xf = &xfv; }
        switch (o.d.kind) {
            case FTP_CONV1D: case FTP_CONV2D: case FTP_FC: {
                const double fl = 2.0 * Mout * o.g.kh * o.g.kw * o.C * o.Co;
                if (m->cfg.precision == FTP_FP32) {
                    Scope sc(m, st, K_CONV_FWD_F32, u, i, 0, (o.in_elems + o.out_elems + o.w_cnt) * 4.0, fl);
                    const bool tc = is_pointwise_op(o) && o.d.kind != FTP_FC && tc32_supported((int)Mout, o.Co, o.C, in, ar.wt + o.w_off, out, nullptr) &&
                                    tc32_gemm((const float*)in, ar.wt + o.w_off, ar.wtl + o.w_off, nullptr, (float*)out, m->red_scratch, (int)Mout, o.Co, o.C,
                                              m->tc_err, st, stats_req, xf);
                    FTP_REQUIRE(tc || !xf, FTP_ECUDA, "forward: op %d: the tensor-core product that applies the preceding batch norm could not be launched", i);
                    if (!tc) next_ps.entries = 0;
                    if (tc && sc.slot) sc.slot->rec.kernel = K_TC32_FWD;
                    const bool stem = !tc && o.d.act == FTP_ACT_NONE && o.b_off < 0 && stem_conv_fwd<float>((const float*)in, ar.w + o.w_off, (float*)out, o.g, st);
                    if (!tc && !stem) conv_fwd_f32((const float*)in, ar.w + o.w_off, o.b_off >= 0 ? ar.w + o.b_off : nullptr, (float*)out, m->red_scratch, o.g, o.d.act, st);
                } else if constexpr (!std::is_same<T, float>::value) {
                    if (o.d.kind == FTP_FC) {           // the classifier runs in float on a widened copy of its input
                        Scope sc(m, st, K_CONV_FWD_F32, u, i, 0, o.in_elems * 2.0 + (o.out_elems + o.w_cnt) * 4.0, fl, 2);
                        bf16_to_f32((const T*)in, m->fc_in, o.in_elems, st);
                        conv_fwd_f32(m->fc_in, ar.w + o.w_off, o.b_off >= 0 ? ar.w + o.b_off : nullptr, (float*)out, m->red_scratch, o.g, o.d.act, st);
                    } else {
                        Scope sc(m, st, K_GEMM_BF16_FWD, u, i, 0, (o.in_elems + o.out_elems + o.w_cnt) * 2.0, fl);
                        bool tc = is_pointwise_op(o) && tc_gemm_supported((int)Mout, o.Co, o.C, in, ar.wbt + o.w_off, out, nullptr) &&
                                  tc_gemm_tn((const T*)in, ar.wbt + o.w_off, nullptr, (T*)out, m->red_scratch, (int)Mout, o.Co, o.C, m->tc_err, st);
                        if (!tc && is_3x3_op(o) && tc_conv3x3_supported(o.N, o.H, o.W, o.C, o.Co, in, ar.wbt + o.w_off, out, nullptr))
                            tc = tc_conv3x3((const T*)in, ar.wbt + o.w_off, nullptr, (T*)out, m->red_scratch, o.N, o.H, o.W, o.C, o.Co, 0, m->tc_err, st);
                        if (!tc && sc.slot) sc.slot->rec.kernel = K_CONV_FWD_BF16_SIMT;
                        if (!tc && o.d.act == FTP_ACT_NONE && o.b_off < 0) tc = stem_conv_fwd<T>((const T*)in, ar.wb + o.w_off, (T*)out, o.g, st);
                        if (!tc) conv_fwd_bf16_simt((const T*)in, ar.wb + o.w_off, o.b_off >= 0 ? ar.w + o.b_off : nullptr, (T*)out, o.g, o.d.act, st);
                    }
                }
                break;
            }
            case FTP_DWCONV3x3: {
                Scope sc(m, st, K_DW_FWD, u, i, 0, (o.in_elems + o.out_elems) * es + o.w_cnt * 4.0, 18.0 * o.out_elems);
                dwconv_fwd<T>((const T*)in, ar.w + o.w_off, (T*)out, o.g, st, stats_req, xf);
                break;
            }
            case FTP_BN: {
                const long long Mr = (long long)o.N * o.H * o.W;
                PartialSums ps = have_ps;
                if (ps.entries <= 0) {
                    Scope sc(m, st, K_BN_STATS, u, i, 0, o.in_elems * es, 3.0 * o.in_elems);
                    ps = bn_stats<T>((const T*)in, Mr, o.C, o.fold, m->fold_scratch, st);
                }
                const void* res = nullptr;
                if (o.fused_add) { const int s = m->ops[i + 1].d.residual_src; res = s < first ? act_in : m->cur_out[s]; }
                { Scope sc(m, st, K_BN_FINALIZE, u, i, 0, ps.entries * 2.0 * o.C * 8.0, 0.0);
                  bn_finalize(ps, Mr, o.C, ar.w + o.w_off, ar.w + o.b_off, m->cfg.bn_eps, m->cfg.bn_momentum,
                              ar.run + o.rm_off, ar.run + o.rv_off, o.scale, o.shift, o.mean, o.mean_lo, o.rstd, o.offset, m->fin, st); }
                if (o.defer) { out = const_cast<void*>(in); break; }       // the next op applies it to what it loads
                { Scope sc(m, st, K_BN_APPLY, u, i, 0, (o.in_elems * (res ? 3.0 : 2.0)) * es, 2.0 * o.in_elems);
                  bn_apply<T>((const T*)in, (const T*)res, (T*)out, Mr, o.C, o.fold, o.scale, o.shift, o.mean, o.mean_lo, o.d.act, st); }
                break;
            }
            case FTP_ACT: {
                Scope sc(m, st, K_ACT_FWD, u, i, 0, 2.0 * o.in_elems * es, (double)o.in_elems);
                act_fwd<T>((const T*)in, (T*)out, o.in_elems, o.d.act, st);
                break;
            }
            case FTP_ADD_RESIDUAL: break;            // folded into the preceding BN
            case FTP_MAXPOOL2: {
                Scope sc(m, st, K_MAXPOOL_FWD, u, i, 0, (o.in_elems + o.out_elems) * es, 3.0 * o.out_elems);
                maxpool_fwd<T>((const T*)in, (T*)out, o.N, o.H, o.W, o.C, st);
                break;
            }
            case FTP_GAP: {
                Scope sc(m, st, K_GAP_FWD, u, i, 0, (o.in_elems + o.out_elems) * es, (double)o.in_elems);
                gap_fwd<T>((const T*)in, (T*)out, o.N, o.H * o.W, o.C, st);
                break;
            }
            case FTP_SOFTMAX_CE: {
                Scope sc(m, st, K_SOFTMAX_CE, u, i, 0, 3.0 * o.in_elems * 4.0, 4.0 * o.in_elems, 2);
                softmax_ce((const float*)in, labels, o.N, o.C, m->per_sample, m->dlogits, loss_out, st);
                out = loss_out;
                break;
            }
        }
        m->cur_out[i] = out;
        if (o.fused_add) m->cur_out[i + 1] = out;
        m->fwd_done[i] = 1;
    }
    if (m->unit_events) cudaEventRecord(m->ev_f[b], st);
    return check_launches("forward");
}

// ---- backward of a unit range -----------------------------------------------------------------------------
template <typename T>
// defer_join (the training step): the caller's stream does not wait for the second stream at the end of this range -- the
// backward pass of the next stage does not depend on this stage's weight gradients, only the update does -- and the
// buffers those weight gradients still read stay listed in m->pending; the caller joins once (join_side) before the update.
ftp_status bwd_range(ftp_model* m, int a, int b, const void* grad_out, void* grad_in, bool internal, cudaStream_t st, bool defer_join = false) {
    const int first = m->unit_first[a], last = m->unit_last[b - 1];
    const double es = (double)m->esize;
    for (int i = first; i <= last; ++i)
        FTP_REQUIRE(m->fwd_done[i], FTP_ESTATE, "run_stage_backward: units [%d,%d) have not been run forward", a, b);
    const void* act_in = m->stage_in[first];
    FTP_REQUIRE(act_in, FTP_ESTATE, "run_stage_backward: the last forward did not start at unit %d", a);
    auto gptr = [&](int j) -> void* {
        const int k = m->ops[j].galias;
        if (k == last && grad_out) return const_cast<void*>(grad_out);
        const int s = m->ops[k].gslot;
        return s == -2 ? (void*)m->dlogits : m->slots[s];
    };
    // Weight gradients feed nothing but the update, so they leave the chain of input gradients: each runs on the second
    // stream after the kernel that produced its output gradient, and the main stream waits for it only before it
    // overwrites the buffer that the weight gradient reads (and once at the end).  Per-unit timing and tracing keep
    // everything on one stream.
    const bool side_on = m->overlap && !m->unit_events && !m->trace;
    std::vector<SidePending>& pending = m->pending;
    struct Join {                                            // the second stream always rejoins the caller's stream, here or in join_side
        ftp_model* m; cudaStream_t st; bool used, deferred;
        ~Join() {
            if (used && deferred) { m->side_unjoined = true; return; }
            if ((used || m->side_unjoined) && cudaEventRecord(m->ev_side.back(), m->side) == cudaSuccess) cudaStreamWaitEvent(st, m->ev_side.back(), 0);
            m->side_unjoined = false;
            m->pending.clear();
        }
    } join{m, st, false, false};
    auto fork = [&](int i) -> cudaStream_t {                 // stream for the weight gradient of operation i
        if (!side_on) return st;
        cudaEventRecord(m->ev_fork[i], st);
        cudaStreamWaitEvent(m->side, m->ev_fork[i], 0);
        join.used = true;
        return m->side;
    };
    auto forked = [&](int i, const void* read) {             // after the launches: remember which buffer they read
        if (!side_on) return;
        cudaEventRecord(m->ev_side[i], m->side);
        pending.push_back({read, m->ev_side[i]});
    };
    auto before_write = [&](const void* buf) {               // main stream is about to overwrite buf
        for (size_t k = 0; k < pending.size();)
            if (pending[k].buf == buf) { cudaStreamWaitEvent(st, pending[k].done, 0); pending.erase(pending.begin() + k); }
            else ++k;
    };
    PartialSums bwd_sums{nullptr, 0, 1};                     // sums of a batch norm's backward pass left by the kernel that produced its output gradient
    int bwd_sums_for = -1;                                   // ... and the batch norm they belong to
    for (int i = last; i >= first; --i) {
        Op& o = m->ops[i];
        const int u = o.d.unit;
        if (m->unit_events && i == m->unit_last[u]) cudaEventRecord(m->ev_b[u + 1], st);
        if (o.d.kind == FTP_SOFTMAX_CE || o.d.kind == FTP_ADD_RESIDUAL) continue;   // dlogits were written by the forward
        const void* in = (i == first) ? act_in : m->cur_out[i - 1];
        const void* go = gptr(i);
        void* gi = nullptr;
        if (i == first) gi = grad_in ? grad_in : ((internal && first > 0) ? m->slots[m->ops[first - 1].gslot] : nullptr);
        else gi = gptr(i - 1);
        const void* addend = o.addend_of >= 0 ? gptr(o.addend_of) : nullptr;
        const Arena& ar = m->arena[m->owner[u]];
        float* gr = m->grad;
        const long long Mout = (long long)o.N * o.Ho * o.Wo;
        if (gi) before_write(gi);
        BnXform xfv{nullptr, nullptr, nullptr, 0.f, 0.f};        // `in` is the input of a deferred batch norm: the weight gradient normalises as it loads
        const BnXform* xf = nullptr;
        if (i > first && m->ops[i - 1].defer) { const Op& bn = m->ops[i - 1]; xfv = make_xform(bn.mean, bn.scale, bn.offset, bn.d.act); xf = &xfv; }
        switch (o.d.kind) {
            case FTP_CONV1D: case FTP_CONV2D: case FTP_FC: {
                const double fl = 2.0 * Mout * o.g.kh * o.g.kw * o.C * o.Co;
                if (m->cfg.precision == FTP_FP32 || o.d.kind == FTP_FC) {
                    const bool widened = m->cfg.precision != FTP_FP32;        // classifier of a bf16 model: float on widened copies
                    FTP_REQUIRE(!(widened && addend), FTP_EUNSUPPORTED, "a residual source feeding the classifier is not supported in bf16 models");
                    const float* x = widened ? m->fc_in : (const float*)in;
                    const float* d = (const float*)go;
                    if (o.d.act != FTP_ACT_NONE || o.b_off >= 0) {
                        float* dpre = o.d.act != FTP_ACT_NONE ? (float*)m->dpre : nullptr;
                        if (dpre) before_write(dpre);
                        Scope sc(m, st, K_ACT_BIAS_BWD, u, i, 1, o.out_elems * 4.0 * (dpre ? 3.0 : 1.0), (double)o.out_elems, o.b_off >= 0 ? 2 : 1);
                        act_bias_bwd<float>(d, (const float*)m->cur_out[i], dpre, Mout, o.Co, o.d.act, o.fold, m->fold_scratch,
                                            o.b_off >= 0 ? gr + o.b_off : nullptr, m->fin, st);
                        if (dpre) d = dpre;
                    }
                    const cudaStream_t ws = fork(i);                 // forked here: the weight gradient depends on nothing after this point
                    auto weight_gradient = [&]() -> ftp_status {
                      Scope sc(m, st, K_CONV_WGRAD_F32, u, i, 1, (o.in_elems + o.out_elems + o.w_cnt) * 4.0, fl, 2);
                      float* rs = ws == st ? m->red_scratch : m->red_side;
                      const bool tc = is_pointwise_op(o) && tc32_supported((int)Mout, o.Co, o.C, x, d, gr + o.w_off, nullptr) &&
                                      tc32_wgrad(x, d, gr + o.w_off, rs, Mout, o.C, o.Co, m->tc_err, ws, xf);
                      FTP_REQUIRE(tc || !xf, FTP_ECUDA, "backward: op %d: the tensor-core weight gradient that applies the preceding batch norm could not be launched", i);
                      if (tc && sc.slot) sc.slot->rec.kernel = K_TC32_WGRAD;
                      const bool stem = !tc && !widened && o.d.act == FTP_ACT_NONE && o.b_off < 0 && stem_conv_wgrad<float>(x, d, gr + o.w_off, rs, o.g, ws);
                      if (!tc && !stem) conv_wgrad_f32(x, d, gr + o.w_off, rs, o.g, ws);
                      forked(i, d);
                      return FTP_OK; };
                    { const ftp_status ws_s = weight_gradient(); if (ws_s != FTP_OK) return ws_s; }
                    if (gi) {
                        Scope sc(m, st, K_CONV_DGRAD_F32, u, i, 1, (o.in_elems * (addend ? 2.0 : 1.0) + o.out_elems + o.w_cnt) * 4.0, fl, widened ? 2 : 1);
                        // dx[M, cin] = dy[M, cout] * w[cin][cout]^T: the weights as they lie are the K-major B operand
                        const bool tc = !widened && is_pointwise_op(o) && tc32_supported((int)Mout, o.C, o.Co, d, ar.w + o.w_off, gi, addend) &&
                                        tc32_gemm(d, ar.w + o.w_off, ar.wl + o.w_off, (const float*)addend, (float*)gi, m->red_scratch, (int)Mout, o.C, o.Co,
                                                  m->tc_err, st);
                        if (tc && sc.slot) sc.slot->rec.kernel = K_TC32_DGRAD;
                        if (!tc) conv_dgrad_f32(d, ar.w + o.w_off, widened ? nullptr : (const float*)addend, widened ? m->fc_din : (float*)gi, m->red_scratch, o.g, st);
                        if (widened) f32_to_bf16(m->fc_din, (__nv_bfloat16*)gi, o.in_elems, st);
                    }
                } else if constexpr (!std::is_same<T, float>::value) {
                    const T* d = (const T*)go;
                    if (o.d.act != FTP_ACT_NONE || o.b_off >= 0) {
                        T* dpre = o.d.act != FTP_ACT_NONE ? (T*)m->dpre : nullptr;
                        if (dpre) before_write(dpre);
                        Scope sc(m, st, K_ACT_BIAS_BWD, u, i, 1, o.out_elems * 2.0 * (dpre ? 3.0 : 1.0), (double)o.out_elems, o.b_off >= 0 ? 2 : 1);
                        act_bias_bwd<T>(d, (const T*)m->cur_out[i], dpre, Mout, o.Co, o.d.act, o.fold, m->fold_scratch,
                                        o.b_off >= 0 ? gr + o.b_off : nullptr, m->fin, st);
                        if (dpre) d = dpre;
                    }
                    const cudaStream_t ws = fork(i);                 // forked here: the weight gradient depends on nothing after this point
                    auto weight_gradient = [&]() {
                      Scope sc(m, st, K_GEMM_BF16_WGRAD, u, i, 1, (o.in_elems + o.out_elems) * 2.0 + o.w_cnt * 4.0, fl, 2);
                      float* rs = ws == st ? m->red_scratch : m->red_side;
                      int splits = 0;
                      if (is_pointwise_op(o) && tc_gemm_supported((int)Mout, o.Co, o.C, in, d, gr + o.w_off, nullptr))
                          splits = tc_wgrad((const T*)in, d, gr + o.w_off, rs, Mout, o.C, o.Co, m->tc_err, ws);
                      if (splits == 0 && is_3x3_op(o) && o.C % 8 == 0 && tc_conv3x3_supported(o.N, o.H, o.W, 64, o.Co, in, d, gr + o.w_off, nullptr))
                          splits = tc_wgrad3x3((const T*)in, d, gr + o.w_off, rs, o.N, o.H, o.W, o.C, o.Co, m->tc_err, ws);
                      if (splits > 1) split_reduce_f32(rs, splits, o.w_cnt, gr + o.w_off, ws);
                      if (splits == 0) {
                          if (sc.slot) sc.slot->rec.kernel = K_CONV_WGRAD_BF16_SIMT;
                          const bool stem = o.d.act == FTP_ACT_NONE && o.b_off < 0 && stem_conv_wgrad<T>((const T*)in, d, gr + o.w_off, rs, o.g, ws);
                          if (!stem) conv_wgrad_bf16_simt((const T*)in, d, gr + o.w_off, rs, o.g, ws);
                      }
                      forked(i, d); };
                    weight_gradient();
                    if (gi) {
                        Scope sc(m, st, K_GEMM_BF16_DGRAD, u, i, 1, (o.in_elems * (addend ? 2.0 : 1.0) + o.out_elems + o.w_cnt) * 2.0, fl);
                        // dx[M, cin] = dy[M, cout] * w[cin][cout]^T: the canonical weight layout already has K = cout contiguous
                        bool tc = is_pointwise_op(o) && tc_gemm_supported((int)Mout, o.C, o.Co, d, ar.wb + o.w_off, gi, addend) &&
                                  tc_gemm_tn(d, ar.wb + o.w_off, (const T*)addend, (T*)gi, m->red_scratch, (int)Mout, o.C, o.Co, m->tc_err, st);
                        if (!tc && is_3x3_op(o) && tc_conv3x3_supported(o.N, o.H, o.W, o.Co, o.C, d, ar.wb + o.w_off, gi, addend))
                            tc = tc_conv3x3(d, ar.wb + o.w_off, (const T*)addend, (T*)gi, m->red_scratch, o.N, o.H, o.W, o.Co, o.C, 1, m->tc_err, st);
                        if (!tc && sc.slot) sc.slot->rec.kernel = K_CONV_DGRAD_BF16_SIMT;
                        if (!tc) conv_dgrad_bf16_simt(d, ar.wb + o.w_off, (const T*)addend, (T*)gi, o.g, st);
                    }
                }
                break;
            }
            case FTP_DWCONV3x3: {
                if (gi && (o.g.stride == 1 || o.g.stride == 2)) {   // one pass over dy gives the input gradient and the weight gradient
                    Scope sc(m, st, K_DW_DGRAD, u, i, 1, (o.in_elems * (addend ? 3.0 : 2.0) + o.out_elems) * es + 2.0 * o.w_cnt * 4.0, 36.0 * o.out_elems, 2);
                    // ... and, when the input is what a deferred batch norm read, the sums of that batch norm's backward pass
                    bwd_sums.entries = 0;
                    BnBwdSumsReq sreq{nullptr, m->fold_scratch, &bwd_sums};
                    const BnBwdSumsReq* sums = nullptr;
                    if (xf && m->bwd_sums_on) { sreq.rstd = m->ops[i - 1].rstd; sums = &sreq; }
                    // the second pass over the blocks' weight-gradient partials feeds only the update: second stream, its own buffers in turn
                    const bool fin_side = side_on && m->dw_fin_side;
                    float* part = m->red_scratch;
                    if (fin_side) { part = m->dw_part[m->dw_rot]; m->dw_rot = (m->dw_rot + 1) % 4; before_write(part); }
                    if (dwconv_bwd_fused<T>((const T*)in, (const T*)go, ar.w + o.w_off, (const T*)addend, (T*)gi, gr + o.w_off, part, o.g, fin_side ? m->fin_side : m->fin,
                                            st, xf, sums, fin_side ? m->side : st, m->ev_fork[i])) {
                        if (fin_side) { join.used = true; forked(i, part); }
                        bwd_sums_for = bwd_sums.entries > 0 ? i - 1 : -1;
                        break;
                    }
                }
                { Scope sc(m, st, K_DW_WGRAD, u, i, 1, (o.in_elems + o.out_elems) * es + o.w_cnt * 4.0, 18.0 * o.out_elems, 2);
                  const cudaStream_t ws = fork(i);
                  dwconv_wgrad<T>((const T*)in, (const T*)go, gr + o.w_off, ws == st ? m->red_scratch : m->red_side, o.g, ws == st ? m->fin : m->fin_side, ws, xf);
                  forked(i, go); }
                if (gi) {
                    Scope sc(m, st, K_DW_DGRAD, u, i, 1, (o.in_elems * (addend ? 2.0 : 1.0) + o.out_elems) * es + o.w_cnt * 4.0, 18.0 * o.out_elems);
                    dwconv_dgrad<T>((const T*)go, ar.w + o.w_off, (const T*)addend, (T*)gi, o.g, st);
                }
                break;
            }
            case FTP_BN: {
                const long long Mr = (long long)o.N * o.H * o.W;
                PartialSums ps;
                const bool premasked = bwd_sums_for == i;          // the producer of `go` masked it and left the sums
                bwd_sums_for = -1;
                if (premasked) ps = bwd_sums;
                else {
                  Scope sc(m, st, K_BN_BWD_REDUCE, u, i, 1, 2.0 * o.in_elems * es, 8.0 * o.in_elems);
                  ps = bn_bwd_reduce<T>((const T*)go, (const T*)in, Mr, o.C, o.fold, o.scale, o.shift, o.mean, o.mean_lo, o.rstd, o.d.act, m->fold_scratch, st); }
                { Scope sc(m, st, K_BN_BWD_FINALIZE, u, i, 1, ps.entries * 2.0 * o.C * 8.0, 0.0);
                  bn_bwd_finalize(ps, Mr, o.C, ar.w + o.w_off, o.rstd, gr + o.w_off, gr + o.b_off, o.coef, m->fin, st); }
                if (gi) {
                    Scope sc(m, st, K_BN_BWD_APPLY, u, i, 1, (addend ? 4.0 : 3.0) * o.in_elems * es, 8.0 * o.in_elems);
                    bn_bwd_apply<T>((const T*)go, (const T*)in, (const T*)addend, (T*)gi, Mr, o.C, o.fold, o.scale, o.shift, o.mean, o.mean_lo, o.rstd, o.coef,
                                    premasked ? FTP_ACT_NONE : o.d.act, st);
                }
                break;
            }
            case FTP_ACT:
                if (gi) {
                    Scope sc(m, st, K_ACT_BWD, u, i, 1, (addend ? 4.0 : 3.0) * o.in_elems * es, (double)o.in_elems);
                    act_bwd<T>((const T*)go, (const T*)in, (const T*)addend, (T*)gi, o.in_elems, o.d.act, st);
                }
                break;
            case FTP_MAXPOOL2:
                FTP_REQUIRE(!addend, FTP_EUNSUPPORTED, "a residual source feeding a max-pool is not supported");
                if (gi) {
                    Scope sc(m, st, K_MAXPOOL_BWD, u, i, 1, (2.0 * o.in_elems + o.out_elems) * es, 4.0 * o.out_elems);
                    maxpool_bwd<T>((const T*)go, (const T*)in, (T*)gi, o.N, o.H, o.W, o.C, st);
                }
                break;
            case FTP_GAP:
                FTP_REQUIRE(!addend, FTP_EUNSUPPORTED, "a residual source feeding a global pool is not supported");
                if (gi) {
                    Scope sc(m, st, K_GAP_BWD, u, i, 1, (o.in_elems + o.out_elems) * es, (double)o.in_elems);
                    gap_bwd<T>((const T*)go, (T*)gi, o.N, o.H * o.W, o.C, st);
                }
                break;
        }
    }
    if (m->unit_events) cudaEventRecord(m->ev_b[a], st);
    const ftp_status launched = check_launches("backward");
    join.deferred = defer_join && launched == FTP_OK;
    return launched;
}

ftp_status check_range(const ftp_model* m, int a, int b, const char* who) {
    FTP_REQUIRE(m, FTP_EINVAL, "%s: null model", who);
    FTP_REQUIRE(a >= 0 && b <= m->L && a < b, FTP_EINVAL, "%s: need 0 <= a < b <= L (a=%d, b=%d, L=%d)", who, a, b, m->L);
    return FTP_OK;
}

// the caller's stream waits for everything the second stream was given by ranges that left without joining
void join_side(ftp_model* m, cudaStream_t st) {
    if (m->side_unjoined && cudaEventRecord(m->ev_side.back(), m->side) == cudaSuccess) cudaStreamWaitEvent(st, m->ev_side.back(), 0);
    m->side_unjoined = false;
    m->pending.clear();
}

ftp_status sgd_range(ftp_model* m, int a, int b, float lr, float* snap_dev, float* snap_host, cudaStream_t st) {
    const float mu = m->cfg.momentum, wd = m->cfg.weight_decay;
    int u = a;
    while (u < b) {
        int v = u + 1;
        while (v < b && m->owner[v] == m->owner[u] && m->mom_init[v] == m->mom_init[u]) ++v;
        const long long off = m->unit_p_off[u];
        const long long cnt = m->unit_p_off[v - 1] + m->unit_p_cnt[v - 1] - off;
        if (cnt > 0) {
            const Arena& ar = m->arena[m->owner[u]];
            const long long rel = off - m->unit_p_off[a];
            Scope sc(m, st, K_SGD, u, -1, 2, cnt * (mu != 0.f ? (m->mom_init[u] ? 20.0 : 16.0) : 12.0) + (ar.wb ? 2.0 * cnt : 0.0) +
                     (snap_dev ? 4.0 * cnt : 0.0) + (snap_host ? 4.0 * cnt : 0.0), 6.0 * cnt);
            sgd_update(ar.w + off, m->grad + off, mu != 0.f ? ar.m + off : nullptr, cnt, lr, mu, wd, m->mom_init[u] ? 0 : 1,
                       ar.wb ? ar.wb + off : nullptr, ar.wl ? ar.wl + off : nullptr, snap_dev ? snap_dev + rel : nullptr,
                       snap_host ? snap_host + rel : nullptr, st);
        }
        for (int k = u; k < v; ++k) m->mom_init[k] = 1;
        u = v;
    }
    refresh_transposed(m, a, b, st);
    return check_launches("sgd_step");
}

template <typename T>
ftp_status train_step_t(ftp_model* m, const void* x, const int32_t* labels, float lr, cudaStream_t st) {
    const void* act = x;
    const bool timing = m->stage_timing && (int)m->ev_sf.size() > m->n_stages;
    if (timing) m->timed_stages = 0;
    for (int s = 0; s < m->n_stages; ++s) {
        const int a = m->points[s], b = m->points[s + 1];
        if (timing) cudaEventRecord(m->ev_sf[s], st);
        ftp_status r = fwd_range<T>(m, a, b, act, nullptr, b == m->L ? labels : nullptr, b == m->L ? m->loss_dev : nullptr, st);
        if (r != FTP_OK) return r;
        act = m->cur_out[m->unit_last[b - 1]];
    }
    if (timing) cudaEventRecord(m->ev_sf[m->n_stages], st);
    for (int s = m->n_stages - 1; s >= 0; --s) {
        if (timing) cudaEventRecord(m->ev_sb[s + 1], st);
        // stage timing wants each stage's weight gradients inside its own interval: those runs join per stage
        ftp_status r = bwd_range<T>(m, m->points[s], m->points[s + 1], nullptr, nullptr, true, st, !timing && m->defer_join);
        if (r != FTP_OK) { join_side(m, st); return r; }
    }
    join_side(m, st);
    if (timing) { cudaEventRecord(m->ev_sb[0], st); m->timed_stages = m->n_stages; }
    for (int s = 0; s < m->n_stages; ++s) {
        ftp_status r = sgd_range(m, m->points[s], m->points[s + 1], lr, nullptr, nullptr, st);
        if (r != FTP_OK) return r;
    }
    return FTP_OK;
}

// The tensor-core kernels bound every wait; one that runs out leaves a code in the device word tc_err.  Every call
// that launches such kernels queues a copy of that word into pinned memory behind its launches (no synchronisation),
// and every later call looks at the copy first: a non-zero code is reported as FTP_ETIMEOUT from then on, until
// ftp_check_device_status reads and clears the word.
int pinned_status(const ftp_model* m) {
    int code;
    std::memcpy(&code, const_cast<const float*>(m->pinned) + 2, 4);
    return code;
}
ftp_status pending_status(const ftp_model* m, const char* who) {
    const int code = pinned_status(m);
    FTP_REQUIRE(code == 0, FTP_ETIMEOUT, "%s: a bounded wait inside an earlier tensor-core kernel ran out (code %d): results since then are invalid; "
                "ftp_check_device_status clears the condition", who, code);
    return FTP_OK;
}
void queue_status(ftp_model* m, cudaStream_t st) { cudaMemcpyAsync(m->pinned + 2, m->tc_err, 4, cudaMemcpyDeviceToHost, st); }

// Synchronising read of the device word; clears it when set.
ftp_status read_device_status(ftp_model* m, cudaStream_t st, const char* who) {
    CUDA_OK(cudaMemcpyAsync(m->pinned + 1, m->tc_err, 4, cudaMemcpyDeviceToHost, st));
    CUDA_OK(cudaStreamSynchronize(st));
    int code;
    std::memcpy(&code, m->pinned + 1, 4);
    if (code == 0) code = pinned_status(m);
    if (code == 0) return FTP_OK;
    CUDA_OK(cudaMemsetAsync(m->tc_err, 0, 4, st));
    CUDA_OK(cudaStreamSynchronize(st));
    std::memset(m->pinned + 1, 0, 8);
    return fail(FTP_ETIMEOUT, "%s: a bounded wait inside a tensor-core kernel ran out (code %d); the tensors written since are invalid, the condition is now cleared", who, code);
}

}  // namespace

// ================================== C ABI ===========================================================

extern "C" ftp_status ftp_workspace_bytes(const ftp_layer_desc* layers, int32_t n, const ftp_model_cfg* cfg, size_t* dev_bytes,
                                          size_t* pinned_bytes) {
    FTP_REQUIRE(dev_bytes && pinned_bytes, FTP_EINVAL, "workspace_bytes: null output");
    ftp_model m{};
    ftp_status s = plan_ops(layers, n, cfg, m);
    if (s != FTP_OK) return s;
    return layout(m, nullptr, dev_bytes, pinned_bytes);
}

extern "C" ftp_status ftp_build_model(const ftp_layer_desc* layers, int32_t n, const ftp_model_cfg* cfg, void* dev_ws, size_t dev_bytes,
                                      void* pinned_ws, size_t pinned_bytes, ftp_model** out) {
    FTP_REQUIRE(out && dev_ws && pinned_ws, FTP_EINVAL, "build_model: null argument");
    FTP_REQUIRE((reinterpret_cast<uintptr_t>(dev_ws) & 255) == 0, FTP_ERANGE, "build_model: the device workspace must be 256-byte aligned");
    ftp_model* m = new (std::nothrow) ftp_model{};
    FTP_REQUIRE(m, FTP_ENOMEM, "build_model: out of host memory");
    ftp_status s = plan_ops(layers, n, cfg, *m);
    size_t need = 0, pneed = 0;
    if (s == FTP_OK) s = layout(*m, (char*)dev_ws, &need, &pneed);
    if (s == FTP_OK && (need > dev_bytes || pneed > pinned_bytes))
        s = fail(FTP_ENOMEM, "build_model: workspace too small (need %zu device and %zu pinned bytes)", need, pneed);
    if (s != FTP_OK) { delete m; return s; }
    m->pinned = (float*)pinned_ws; m->pinned_bytes = pinned_bytes;
    m->ws_base = (char*)dev_ws;
    for (size_t off : m->guards)
        if (cudaMemset(m->ws_base + off, kGuardByte, kGuardBytes) != cudaSuccess) {
            const ftp_status e = fail(FTP_ECUDA, "build_model: filling the guard zones failed: %s", cudaGetErrorString(cudaGetLastError()));
            delete m;
            return e;
        }
    std::memset(m->pinned, 0, 16);                            // loss, status words
    if (cudaMemset(m->fin.counters, 0, m->fin_counter_bytes) != cudaSuccess || cudaMemset(m->fin_side.counters, 0, m->fin_counter_bytes) != cudaSuccess ||
        cudaMemset(m->tc_err, 0, 256) != cudaSuccess) {     // ticket counters start at zero
        const ftp_status e = fail(FTP_ECUDA, "build_model: clearing the ticket counters failed: %s", cudaGetErrorString(cudaGetLastError()));
        delete m;
        return e;
    }
    if (cudaMemcpy(m->tp_dev, m->tp_host.data(), m->tp_host.size() * sizeof(TransposeEntryDev), cudaMemcpyHostToDevice) != cudaSuccess) {
        const ftp_status e = fail(FTP_ECUDA, "build_model: uploading the transposition table failed: %s", cudaGetErrorString(cudaGetLastError()));
        delete m;
        return e;
    }
    {   // second stream and its fork / join events: one pair per operation, created here so that nothing is created inside a stream capture
        const char* e = std::getenv("FTP_OVERLAP");
        m->overlap = !(e && std::strcmp(e, "0") == 0);
        {   // One join before the update instead of one per stage: measured 1.403 -> 1.377 ms on VGG-16 (few, long weight
            // gradients), but 3.254 -> 3.280 ms and 4.97 -> 5.01 ms on the MobileNetV2 configurations, whose many short weight
            // gradients then pile up beside the large early layers of the next stage.  Default: only for networks without
            // depthwise convolutions; FTP_DEFER_JOIN=0 / 1 overrides.
            bool has_dw = false;
            for (const Op& o : m->ops) has_dw = has_dw || o.d.kind == FTP_DWCONV3x3;
            const char* df = std::getenv("FTP_DW_FIN_SIDE");
            m->dw_fin_side = !(df && std::strcmp(df, "0") == 0);
            const char* dj = std::getenv("FTP_DEFER_JOIN");
            m->defer_join = dj ? std::strcmp(dj, "0") != 0 : !has_dw;
        }
        const char* ps = std::getenv("FTP_PRODUCER_STATS");          // 0: batch-norm statistics always by their own kernel (A/B measurements)
        m->producer_stats = !(ps && std::strcmp(ps, "0") == 0);
        // FTP_BWD_SUMS: 0 = the first pass of every batch-norm backward by its own kernel, 1 = from the depthwise backward
        // kernel where it can give them.  Default: 1 in float models, 0 in bf16 models (the kernel with the sums inside
        // took longer there than the reduction pass it saves).
        const char* bs = std::getenv("FTP_BWD_SUMS");
        m->bwd_sums_on = bs ? std::strcmp(bs, "0") != 0 : m->cfg.precision == FTP_FP32;
        bool ok = cudaStreamCreateWithFlags(&m->side, cudaStreamNonBlocking) == cudaSuccess;
        for (size_t i = 0; ok && i <= m->ops.size(); ++i) {
            cudaEvent_t a = nullptr, b = nullptr;
            ok = cudaEventCreateWithFlags(&a, cudaEventDisableTiming) == cudaSuccess && cudaEventCreateWithFlags(&b, cudaEventDisableTiming) == cudaSuccess;
            if (a) m->ev_fork.push_back(a);
            if (b) m->ev_side.push_back(b);
        }
        if (!ok) {
            const ftp_status er = fail(FTP_ECUDA, "build_model: creating the second stream failed: %s", cudaGetErrorString(cudaGetLastError()));
            ftp_destroy_model(m);
            return er;
        }
    }
    m->owner.assign(m->L, 0);
    m->points = {0, m->L};
    m->n_stages = 1;
    m->worker.assign(1, 0);
    m->mom_init.assign(m->L, 0);
    m->stage_in.assign(m->ops.size(), nullptr);
    m->cur_out.assign(m->ops.size(), nullptr);
    m->fwd_done.assign(m->ops.size(), 0);
    m->trace = false; m->tr_used = 0; m->unit_events = false;
    *out = m;
    return FTP_OK;
}

extern "C" void ftp_destroy_model(ftp_model* m) {
    if (!m) return;
    for (auto& t : m->tr) { cudaEventDestroy(t.e0); cudaEventDestroy(t.e1); }
    for (auto e : m->ev_f) cudaEventDestroy(e);
    for (auto e : m->ev_b) cudaEventDestroy(e);
    for (auto e : m->ev_sf) cudaEventDestroy(e);
    for (auto e : m->ev_sb) cudaEventDestroy(e);
    for (auto e : m->ev_fork) cudaEventDestroy(e);
    for (auto e : m->ev_side) cudaEventDestroy(e);
    if (m->side) cudaStreamDestroy(m->side);
    delete m;
}

extern "C" ftp_status ftp_num_units(const ftp_model* m, int32_t* L) {
    FTP_REQUIRE(m && L, FTP_EINVAL, "num_units: null argument");
    *L = m->L;
    return FTP_OK;
}

extern "C" ftp_status ftp_unit_param_span(const ftp_model* m, int32_t unit, int64_t* offset, int64_t* count) {
    FTP_REQUIRE(m && offset && count, FTP_EINVAL, "unit_param_span: null argument");
    FTP_REQUIRE(unit >= 0 && unit < m->L, FTP_ERANGE, "unit_param_span: unit %d out of range", unit);
    *offset = m->unit_p_off[unit]; *count = m->unit_p_cnt[unit];
    return FTP_OK;
}

extern "C" ftp_status ftp_unit_state_span(const ftp_model* m, int32_t unit, int64_t* offset, int64_t* count) {
    FTP_REQUIRE(m && offset && count, FTP_EINVAL, "unit_state_span: null argument");
    FTP_REQUIRE(unit >= 0 && unit < m->L, FTP_ERANGE, "unit_state_span: unit %d out of range", unit);
    *offset = m->unit_s_off[unit]; *count = m->unit_s_cnt[unit];
    return FTP_OK;
}

extern "C" ftp_status ftp_unit_output_shape(const ftp_model* m, int32_t unit, int32_t shape[4], int64_t* bytes) {
    FTP_REQUIRE(m && shape && bytes, FTP_EINVAL, "unit_output_shape: null argument");
    FTP_REQUIRE(unit >= 0 && unit < m->L, FTP_ERANGE, "unit_output_shape: unit %d out of range", unit);
    const Op& o = m->ops[m->unit_last[unit]];
    if (o.d.kind == FTP_SOFTMAX_CE) { shape[0] = shape[1] = shape[2] = shape[3] = 1; *bytes = 4; return FTP_OK; }
    shape[0] = o.N; shape[1] = o.Ho; shape[2] = o.Wo; shape[3] = o.Co;
    *bytes = o.out_elems * (o.out_f32 ? 4 : m->esize);
    return FTP_OK;
}

static ftp_status tensor_ptr(const ftp_model* m, int which, int unit, int64_t count, float** p, const char* who) {
    FTP_REQUIRE(m, FTP_EINVAL, "%s: null model", who);
    FTP_REQUIRE(unit >= 0 && unit < m->L, FTP_ERANGE, "%s: unit %d out of range", who, unit);
    const Arena& ar = m->arena[m->owner[unit]];
    long long want = m->unit_p_cnt[unit];
    switch (which) {
        case FTP_T_WEIGHTS: *p = ar.w + m->unit_p_off[unit]; break;
        case FTP_T_GRADS: *p = m->grad + m->unit_p_off[unit]; break;
        case FTP_T_MOMENTUM: *p = ar.m + m->unit_p_off[unit]; break;
        case FTP_T_STATE: *p = ar.run + m->unit_s_off[unit]; want = m->unit_s_cnt[unit]; break;
        default: return fail(FTP_EINVAL, "%s: unknown tensor selector %d", who, which);
    }
    FTP_REQUIRE(count == want, FTP_ERANGE, "%s: unit %d holds %lld floats, caller passed %lld", who, unit, want, (long long)count);
    return FTP_OK;
}

extern "C" ftp_status ftp_set_tensor(ftp_model* m, int32_t which, int32_t unit, const float* src, int64_t count, int32_t src_is_device,
                                     void* stream) {
    float* dst = nullptr;
    ftp_status s = tensor_ptr(m, which, unit, count, &dst, "set_tensor");
    if (s != FTP_OK) return s;
    if (count == 0) return FTP_OK;
    FTP_REQUIRE(src, FTP_EINVAL, "set_tensor: null source");
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_OK(cudaMemcpyAsync(dst, src, (size_t)count * 4, src_is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, st));
    if (which == FTP_T_WEIGHTS) {
        const Arena& ar = m->arena[m->owner[unit]];
        if (ar.wb) {
            Scope sc(m, st, K_COPY, unit, -1, 2, 6.0 * count, 0.0);
            f32_to_bf16(dst, ar.wb + m->unit_p_off[unit], count, st);
            refresh_transposed(m, unit, unit + 1, st);
        }
        if (ar.wl) {
            Scope sc(m, st, K_COPY, unit, -1, 2, 16.0 * count, 0.0);
            tf32_lo(dst, ar.wl + m->unit_p_off[unit], count, st);
            refresh_transposed(m, unit, unit + 1, st);
        }
        m->mom_init[unit] = 0;
    } else if (which == FTP_T_MOMENTUM) m->mom_init[unit] = 1;
    if (!src_is_device) CUDA_OK(cudaStreamSynchronize(st));
    return check_launches("set_tensor");
}

extern "C" ftp_status ftp_get_tensor(const ftp_model* m, int32_t which, int32_t unit, float* dst, int64_t count, int32_t dst_is_device,
                                     void* stream) {
    float* src = nullptr;
    ftp_status s = tensor_ptr(m, which, unit, count, &src, "get_tensor");
    if (s != FTP_OK) return s;
    if (count == 0) return FTP_OK;
    FTP_REQUIRE(dst, FTP_EINVAL, "get_tensor: null destination");
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_OK(cudaMemcpyAsync(dst, src, (size_t)count * 4, dst_is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost, st));
    if (!dst_is_device) return read_device_status(const_cast<ftp_model*>(m), st, "get_tensor");
    return FTP_OK;
}

extern "C" ftp_status ftp_run_stage_forward(ftp_model* m, int32_t a, int32_t b, const void* act_in, void* act_out, const int32_t* labels,
                                            float* loss_out, void* stream) {
    ftp_status s = check_range(m, a, b, "run_stage_forward");
    if (s == FTP_OK) s = pending_status(m, "run_stage_forward");
    if (s != FTP_OK) return s;
    FTP_REQUIRE(act_in, FTP_EINVAL, "run_stage_forward: null act_in");
    FTP_REQUIRE(a16(act_in) && a16(act_out), FTP_ERANGE, "run_stage_forward: activation buffers must be 16-byte aligned");
    if (b == m->L) FTP_REQUIRE(labels && loss_out && !act_out, FTP_EINVAL, "run_stage_forward: the last stage needs labels and loss_out, and no act_out");
    else FTP_REQUIRE(act_out && !labels && !loss_out, FTP_EINVAL, "run_stage_forward: an inner stage needs act_out and takes no labels");
    cudaStream_t st = (cudaStream_t)stream;
    s = m->cfg.precision == FTP_FP32 ? fwd_range<float>(m, a, b, act_in, act_out, labels, loss_out, st)
                                     : fwd_range<__nv_bfloat16>(m, a, b, act_in, act_out, labels, loss_out, st);
    queue_status(m, st);
    return s;
}

extern "C" ftp_status ftp_run_stage_backward(ftp_model* m, int32_t a, int32_t b, const void* grad_out, void* grad_in, void* stream) {
    ftp_status s = check_range(m, a, b, "run_stage_backward");
    if (s == FTP_OK) s = pending_status(m, "run_stage_backward");
    if (s != FTP_OK) return s;
    if (b == m->L) FTP_REQUIRE(!grad_out, FTP_EINVAL, "run_stage_backward: the last stage takes no grad_out");
    else FTP_REQUIRE(grad_out, FTP_EINVAL, "run_stage_backward: an inner stage needs grad_out");
    FTP_REQUIRE(a == 0 || grad_in, FTP_EINVAL, "run_stage_backward: grad_in is required when a > 0");
    FTP_REQUIRE(a16(grad_out) && a16(grad_in), FTP_ERANGE, "run_stage_backward: gradient buffers must be 16-byte aligned");
    cudaStream_t st = (cudaStream_t)stream;
    s = m->cfg.precision == FTP_FP32 ? bwd_range<float>(m, a, b, grad_out, grad_in, false, st)
                                     : bwd_range<__nv_bfloat16>(m, a, b, grad_out, grad_in, false, st);
    queue_status(m, st);
    return s;
}

extern "C" ftp_status ftp_get_logits(const ftp_model* m, float* dst, int32_t dst_is_device, void* stream) {
    FTP_REQUIRE(m && dst, FTP_EINVAL, "get_logits: null argument");
    const int fc = (int)m->ops.size() - 2;
    FTP_REQUIRE(m->fwd_done[fc] && m->cur_out[fc], FTP_ESTATE, "get_logits: no forward has reached the last unit yet");
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_OK(cudaMemcpyAsync(dst, m->cur_out[fc], (size_t)m->cfg.batch * m->cfg.n_classes * 4,
                            dst_is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost, st));
    if (!dst_is_device) return read_device_status(const_cast<ftp_model*>(m), st, "get_logits");
    return FTP_OK;
}

extern "C" ftp_status ftp_sgd_step(ftp_model* m, int32_t a, int32_t b, float lr, float* snap_dev, float* snap_host, void* stream) {
    ftp_status s = check_range(m, a, b, "sgd_step");
    if (s == FTP_OK) s = pending_status(m, "sgd_step");
    if (s != FTP_OK) return s;
    s = sgd_range(m, a, b, lr, snap_dev, snap_host, (cudaStream_t)stream);
    queue_status(m, (cudaStream_t)stream);
    return s;
}

extern "C" ftp_status ftp_train_step(ftp_model* m, const void* x, const int32_t* labels, int32_t inputs_on_host, float lr, float* loss_host,
                                     void* stream) {
    FTP_REQUIRE(m && x && labels, FTP_EINVAL, "train_step: null argument");
    {
        const ftp_status ps = pending_status(m, "train_step");
        if (ps != FTP_OK) return ps;
    }
    cudaStream_t st = (cudaStream_t)stream;
    const void* xin = x;
    const int32_t* lab = labels;
    if (inputs_on_host) {
        for (int i = 0; i < m->cfg.batch; ++i)
            FTP_REQUIRE(labels[i] >= 0 && labels[i] < m->cfg.n_classes, FTP_ERANGE, "train_step: label %d of sample %d is outside [0, %d)", labels[i], i, m->cfg.n_classes);
        const size_t in_bytes = (size_t)m->cfg.batch * m->cfg.in_h * m->cfg.in_w * m->cfg.in_c * m->esize;
        CUDA_OK(cudaMemcpyAsync(m->input_dev, x, in_bytes, cudaMemcpyHostToDevice, st));
        CUDA_OK(cudaMemcpyAsync(m->labels_dev, labels, (size_t)m->cfg.batch * 4, cudaMemcpyHostToDevice, st));
        xin = m->input_dev; lab = m->labels_dev;
    } else FTP_REQUIRE(a16(x), FTP_ERANGE, "train_step: the input batch must be 16-byte aligned");
    ftp_status s = m->cfg.precision == FTP_FP32 ? train_step_t<float>(m, xin, lab, lr, st) : train_step_t<__nv_bfloat16>(m, xin, lab, lr, st);
    if (s != FTP_OK) return s;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) cap = cudaStreamCaptureStatusNone;
    if (loss_host && cap == cudaStreamCaptureStatusNone) {
        CUDA_OK(cudaMemcpyAsync(m->pinned, m->loss_dev, 4, cudaMemcpyDeviceToHost, st));
        s = read_device_status(m, st, "train_step");
        *loss_host = m->pinned[0];
        return s;
    }
    if (loss_host) CUDA_OK(cudaMemcpyAsync(loss_host, m->loss_dev, 4, cudaMemcpyDeviceToHost, st));    // recorded into the caller's graph
    queue_status(m, st);
    return FTP_OK;
}

// Sec. III-B: every worker measures the bandwidth to its next worker (B_{i,i+1} of Eq. 5).  With all stages on one GPU
// the "links" are copies inside device memory and, towards the central node's host copy, the path to pinned host memory.
extern "C" ftp_status ftp_measure_bandwidth(ftp_model* m, void* pinned_host, size_t bytes, int32_t reps, double* d2d_bytes_per_s,
                                            double* d2h_bytes_per_s, void* stream) {
    FTP_REQUIRE(m && d2d_bytes_per_s && d2h_bytes_per_s, FTP_EINVAL, "measure_bandwidth: null argument");
    FTP_REQUIRE(reps >= 1 && reps <= 1000 && bytes >= 4096, FTP_EINVAL, "measure_bandwidth: reps must be in 1..1000 and bytes at least 4096");
    cudaStream_t st = (cudaStream_t)stream;
    const size_t n = std::min(bytes, m->red_floats * 4);          // the two reduction scratch areas are idle between steps
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    CUDA_OK(cudaEventCreate(&e0));
    if (cudaEventCreate(&e1) != cudaSuccess) { cudaEventDestroy(e0); return fail(FTP_ECUDA, "measure_bandwidth: cudaEventCreate failed"); }
    auto timed = [&](void* dst, const void* src, cudaMemcpyKind kind, double* out) -> ftp_status {
        cudaError_t e = cudaMemcpyAsync(dst, src, n, kind, st);                    // warm-up
        if (e == cudaSuccess) e = cudaEventRecord(e0, st);
        for (int r = 0; r < reps && e == cudaSuccess; ++r) e = cudaMemcpyAsync(dst, src, n, kind, st);
        if (e == cudaSuccess) e = cudaEventRecord(e1, st);
        if (e == cudaSuccess) e = cudaEventSynchronize(e1);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
        if (e != cudaSuccess) return fail(FTP_ECUDA, "measure_bandwidth: %s", cudaGetErrorString(e));
        *out = ms > 0.f ? (double)n * reps / (ms * 1e-3) : 0.0;
        return FTP_OK;
    };
    ftp_status s = timed(m->red_side, m->red_scratch, cudaMemcpyDeviceToDevice, d2d_bytes_per_s);
    *d2h_bytes_per_s = 0.0;
    if (s == FTP_OK && pinned_host) s = timed(pinned_host, m->red_scratch, cudaMemcpyDeviceToHost, d2h_bytes_per_s);
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    return s;
}

extern "C" ftp_status ftp_check_guards(ftp_model* m, int32_t* n_guards, int64_t* first_bad_offset, void* stream) {
    FTP_REQUIRE(m, FTP_EINVAL, "check_guards: null model");
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_OK(cudaStreamSynchronize(st));
    if (n_guards) *n_guards = (int32_t)m->guards.size();
    if (first_bad_offset) *first_bad_offset = -1;
    unsigned char buf[kGuardBytes];
    for (size_t k = 0; k < m->guards.size(); ++k) {
        CUDA_OK(cudaMemcpy(buf, m->ws_base + m->guards[k], kGuardBytes, cudaMemcpyDeviceToHost));
        for (size_t i = 0; i < kGuardBytes; ++i)
            if (buf[i] != kGuardByte) {
                if (first_bad_offset) *first_bad_offset = (int64_t)(m->guards[k] + i);
                return fail(FTP_ESTATE, "check_guards: guard zone %zu of %zu was overwritten at workspace offset %zu: a kernel wrote past the end of the buffer before it",
                            k, m->guards.size(), m->guards[k] + i);
            }
    }
    return FTP_OK;
}

extern "C" ftp_status ftp_check_device_status(ftp_model* m, void* stream) {
    FTP_REQUIRE(m, FTP_EINVAL, "check_device_status: null model");
    return read_device_status(m, (cudaStream_t)stream, "check_device_status");
}

extern "C" ftp_status ftp_debug_set_device_status(ftp_model* m, int32_t code, void* stream) {
    FTP_REQUIRE(m, FTP_EINVAL, "debug_set_device_status: null model");
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_OK(cudaMemcpyAsync(m->tc_err, &code, 4, cudaMemcpyHostToDevice, st));
    CUDA_OK(cudaStreamSynchronize(st));
    return FTP_OK;
}

extern "C" ftp_status ftp_stage_timing_enable(ftp_model* m, int32_t on) {
    FTP_REQUIRE(m, FTP_EINVAL, "stage_timing_enable: null model");
    const size_t need = (size_t)m->cfg.max_stages + 1;
    while (on && m->ev_sf.size() < need) { cudaEvent_t e; CUDA_OK(cudaEventCreate(&e)); m->ev_sf.push_back(e); }
    while (on && m->ev_sb.size() < need) { cudaEvent_t e; CUDA_OK(cudaEventCreate(&e)); m->ev_sb.push_back(e); }
    m->stage_timing = on != 0;
    m->timed_stages = 0;
    return FTP_OK;
}

extern "C" ftp_status ftp_stage_times(ftp_model* m, double* seconds, int32_t* n_stages) {
    FTP_REQUIRE(m && seconds && n_stages, FTP_EINVAL, "stage_times: null argument");
    FTP_REQUIRE(m->timed_stages > 0, FTP_ESTATE, "stage_times: no training step has run since stage timing was switched on");
    const int n = m->timed_stages;
    CUDA_OK(cudaEventSynchronize(m->ev_sb[0]));
    {
        const ftp_status ps = pending_status(m, "stage_times");
        if (ps != FTP_OK) return ps;
    }
    for (int s = 0; s < n; ++s) {
        float f = 0.f, b = 0.f;
        CUDA_OK(cudaEventElapsedTime(&f, m->ev_sf[s], m->ev_sf[s + 1]));
        CUDA_OK(cudaEventElapsedTime(&b, m->ev_sb[s + 1], m->ev_sb[s]));
        seconds[s] = ((double)f + (double)b) * 1e-3;
    }
    *n_stages = n;
    return FTP_OK;
}

extern "C" ftp_status ftp_profile_layers(ftp_model* m, int32_t reps, const void* sample_in, const int32_t* labels, double* fwd_s,
                                         double* bwd_s, int64_t* out_bytes, void* stream) {
    FTP_REQUIRE(m && sample_in && labels && fwd_s && bwd_s && out_bytes, FTP_EINVAL, "profile_layers: null argument");
    FTP_REQUIRE(reps >= 1 && reps <= 1000, FTP_EINVAL, "profile_layers: reps must be in 1..1000");
    FTP_REQUIRE(a16(sample_in), FTP_ERANGE, "profile_layers: the sample batch must be 16-byte aligned");
    {
        const ftp_status ps = pending_status(m, "profile_layers");
        if (ps != FTP_OK) return ps;
    }
    cudaStream_t st = (cudaStream_t)stream;
    const int L = m->L;
    while ((int)m->ev_f.size() < L + 1) { cudaEvent_t e; CUDA_OK(cudaEventCreate(&e)); m->ev_f.push_back(e); }
    while ((int)m->ev_b.size() < L + 1) { cudaEvent_t e; CUDA_OK(cudaEventCreate(&e)); m->ev_b.push_back(e); }
    // keep the BN running statistics: profiling is not training
    for (int u = 0; u < L; ++u)
        if (m->unit_s_cnt[u])
            CUDA_OK(cudaMemcpyAsync(m->state_backup + m->unit_s_off[u], m->arena[m->owner[u]].run + m->unit_s_off[u],
                                    (size_t)m->unit_s_cnt[u] * 4, cudaMemcpyDeviceToDevice, st));
    std::vector<double> f(L, 0.0), bk(L, 0.0);
    ftp_status s = FTP_OK;
    const bool was_tracing = m->trace;
    m->trace = false;
    for (int r = -1; r < reps && s == FTP_OK; ++r) {            // r == -1: untimed warm-up pass
        m->unit_events = r >= 0;
        s = m->cfg.precision == FTP_FP32 ? fwd_range<float>(m, 0, L, sample_in, nullptr, labels, m->loss_dev, st)
                                         : fwd_range<__nv_bfloat16>(m, 0, L, sample_in, nullptr, labels, m->loss_dev, st);
        if (s == FTP_OK)
            s = m->cfg.precision == FTP_FP32 ? bwd_range<float>(m, 0, L, nullptr, nullptr, true, st)
                                             : bwd_range<__nv_bfloat16>(m, 0, L, nullptr, nullptr, true, st);
        if (s != FTP_OK) break;
        if (cudaStreamSynchronize(st) != cudaSuccess) { s = fail(FTP_ECUDA, "profile_layers: stream synchronisation failed"); break; }
        if (r < 0) continue;
        for (int u = 0; u < L; ++u) {
            float ms = 0.f;
            cudaEventElapsedTime(&ms, m->ev_f[u], m->ev_f[u + 1]); f[u] += ms * 1e-3;
            cudaEventElapsedTime(&ms, m->ev_b[u + 1], m->ev_b[u]); bk[u] += ms * 1e-3;
        }
    }
    m->unit_events = false;
    m->trace = was_tracing;
    for (int u = 0; u < L; ++u)
        if (m->unit_s_cnt[u])
            cudaMemcpyAsync(m->arena[m->owner[u]].run + m->unit_s_off[u], m->state_backup + m->unit_s_off[u], (size_t)m->unit_s_cnt[u] * 4,
                            cudaMemcpyDeviceToDevice, st);
    cudaStreamSynchronize(st);
    if (s == FTP_OK) s = read_device_status(m, st, "profile_layers");
    if (s != FTP_OK) return s;
    for (int u = 0; u < L; ++u) {
        fwd_s[u] = f[u] / reps; bwd_s[u] = bk[u] / reps;
        int32_t shp[4];
        ftp_unit_output_shape(m, u, shp, &out_bytes[u]);
    }
    return check_launches("profile_layers");
}

// Everything arena `from` holds of unit u (weights, momentum, running statistics and the derived copies) -> arena `to`.
static ftp_status copy_unit(ftp_model* m, int u, int from_arena, int to_arena, cudaStream_t st) {
    const Arena& from = m->arena[from_arena];
    const Arena& to = m->arena[to_arena];
    const long long po = m->unit_p_off[u], pc = m->unit_p_cnt[u], so = m->unit_s_off[u], sc_ = m->unit_s_cnt[u];
    if (pc) {
        CUDA_OK(cudaMemcpyAsync(to.w + po, from.w + po, (size_t)pc * 4, cudaMemcpyDeviceToDevice, st));
        CUDA_OK(cudaMemcpyAsync(to.m + po, from.m + po, (size_t)pc * 4, cudaMemcpyDeviceToDevice, st));
        if (to.wb) CUDA_OK(cudaMemcpyAsync(to.wb + po, from.wb + po, (size_t)pc * 2, cudaMemcpyDeviceToDevice, st));
        if (to.wbt) CUDA_OK(cudaMemcpyAsync(to.wbt + po, from.wbt + po, (size_t)pc * 2, cudaMemcpyDeviceToDevice, st));
        if (to.wl) {
            CUDA_OK(cudaMemcpyAsync(to.wl + po, from.wl + po, (size_t)pc * 4, cudaMemcpyDeviceToDevice, st));
            CUDA_OK(cudaMemcpyAsync(to.wt + po, from.wt + po, (size_t)pc * 4, cudaMemcpyDeviceToDevice, st));
            CUDA_OK(cudaMemcpyAsync(to.wtl + po, from.wtl + po, (size_t)pc * 4, cudaMemcpyDeviceToDevice, st));
        }
    }
    if (sc_) CUDA_OK(cudaMemcpyAsync(to.run + so, from.run + so, (size_t)sc_ * 4, cudaMemcpyDeviceToDevice, st));
    return FTP_OK;
}

extern "C" ftp_status ftp_set_partition(ftp_model* m, const int32_t* points, int32_t n_stages, int32_t* moved_units, void* stream) {
    FTP_REQUIRE(m && points, FTP_EINVAL, "set_partition: null argument");
    FTP_REQUIRE(n_stages >= 1 && n_stages <= m->cfg.max_stages && n_stages <= m->L, FTP_EINVAL,
                "set_partition: %d stages not in 1..min(max_stages=%d, L=%d)", n_stages, m->cfg.max_stages, m->L);
    FTP_REQUIRE(points[0] == 0 && points[n_stages] == m->L, FTP_EINVAL, "set_partition: points must run from 0 to L");
    for (int i = 0; i < n_stages; ++i) FTP_REQUIRE(points[i] < points[i + 1], FTP_EINVAL, "set_partition: stage %d is empty", i);
    cudaStream_t st = (cudaStream_t)stream;
    int moved = 0;
    std::vector<int32_t> plan(m->L);
    // stages beyond the current worker list are joined by workers whose arenas are idle (lowest first)
    std::vector<int> worker = m->worker;
    worker.resize(std::min<size_t>(worker.size(), (size_t)n_stages));
    for (int a = 0; (int)worker.size() < n_stages && a < m->cfg.max_stages; ++a)
        if (std::find(worker.begin(), worker.end(), a) == worker.end()) worker.push_back(a);
    FTP_REQUIRE((int)worker.size() == n_stages, FTP_ESTATE, "set_partition: no idle arena left for %d stages", n_stages);
    // Phase 1: every stage fetches what Algorithm 1 says it is missing, from the current owner's arena.
    for (int i = 0; i < n_stages; ++i) {
        int32_t n_local = 0;
        ftp_status s = ftp_redistribution_plan(points, n_stages, m->points.data(), m->n_stages, -1, i < m->n_stages ? i : -1, i, plan.data(), &n_local);
        if (s != FTP_OK) return s;
        for (int u = points[i]; u < points[i + 1]; ++u) {
            const int src = plan[u - points[i]];
            if (src < 0) continue;                                   // already local
            ++moved;
            Scope sc(m, st, K_COPY, u, -1, 2, (m->unit_p_cnt[u] * 2 + m->unit_s_cnt[u]) * 8.0, 0.0, 0);
            const ftp_status cs = copy_unit(m, u, m->worker[src], worker[i], st);
            if (cs != FTP_OK) return cs;
        }
    }
    // Phase 2 (commit): only now does the owner table switch; later launches are stream-ordered after the copies.
    for (int i = 0; i < n_stages; ++i)
        for (int u = points[i]; u < points[i + 1]; ++u) m->owner[u] = worker[i];
    m->worker = worker;
    m->points.assign(points, points + n_stages + 1);
    m->n_stages = n_stages;
    std::fill(m->fwd_done.begin(), m->fwd_done.end(), 0);
    if (moved_units) *moved_units = moved;
    return FTP_OK;
}

// ---- asynchronous pipeline training (Sec. III-C): weight versions live in models of the same architecture ----------
static ftp_status same_architecture(const ftp_model* a, const ftp_model* b, const char* who) {
    FTP_REQUIRE(a && b, FTP_EINVAL, "%s: null model", who);
    FTP_REQUIRE(a->L == b->L && a->P == b->P && a->R == b->R && a->cfg.precision == b->cfg.precision && a->unit_p_off == b->unit_p_off &&
                a->unit_s_off == b->unit_s_off, FTP_EINVAL, "%s: the models were not built from the same layer list", who);
    return FTP_OK;
}

// after the float masters of units [a, b) changed: the copies the kernels read (bf16 shadow, tf32 lo part, transposes)
static void refresh_derived(ftp_model* m, int a, int b, cudaStream_t st) {
    for (int u = a; u < b; ++u) {
        const Arena& ar = m->arena[m->owner[u]];
        const long long po = m->unit_p_off[u], pc = m->unit_p_cnt[u];
        if (!pc) continue;
        if (ar.wb) f32_to_bf16(ar.w + po, ar.wb + po, pc, st);
        if (ar.wl) tf32_lo(ar.w + po, ar.wl + po, pc, st);
    }
    refresh_transposed(m, a, b, st);
}

extern "C" ftp_status ftp_sync_units(ftp_model* dst, const ftp_model* src, int32_t a, int32_t b, int32_t what, void* stream) {
    ftp_status s = same_architecture(dst, src, "sync_units");
    if (s == FTP_OK) s = check_range(dst, a, b, "sync_units");
    if (s != FTP_OK) return s;
    FTP_REQUIRE(what > 0 && what < 8, FTP_EINVAL, "sync_units: `what` is a mask of FTP_SYNC_WEIGHTS, FTP_SYNC_MOMENTUM, FTP_SYNC_STATE");
    cudaStream_t st = (cudaStream_t)stream;
    for (int u = a; u < b; ++u) {
        const Arena& to = dst->arena[dst->owner[u]];
        const Arena& from = src->arena[src->owner[u]];
        const long long po = dst->unit_p_off[u], pc = dst->unit_p_cnt[u], so = dst->unit_s_off[u], sc_ = dst->unit_s_cnt[u];
        if ((what & FTP_SYNC_WEIGHTS) && pc) CUDA_OK(cudaMemcpyAsync(to.w + po, from.w + po, (size_t)pc * 4, cudaMemcpyDeviceToDevice, st));
        if ((what & FTP_SYNC_MOMENTUM) && pc) {
            CUDA_OK(cudaMemcpyAsync(to.m + po, from.m + po, (size_t)pc * 4, cudaMemcpyDeviceToDevice, st));
            dst->mom_init[u] = src->mom_init[u];
        }
        if ((what & FTP_SYNC_STATE) && sc_) CUDA_OK(cudaMemcpyAsync(to.run + so, from.run + so, (size_t)sc_ * 4, cudaMemcpyDeviceToDevice, st));
    }
    if (what & FTP_SYNC_WEIGHTS) refresh_derived(dst, a, b, st);
    return check_launches("sync_units");
}

extern "C" ftp_status ftp_sgd_step_from(ftp_model* dst, const ftp_model* grads, int32_t a, int32_t b, float lr, void* stream) {
    ftp_status s = same_architecture(dst, grads, "sgd_step_from");
    if (s == FTP_OK) s = check_range(dst, a, b, "sgd_step_from");
    if (s == FTP_OK) s = pending_status(dst, "sgd_step_from");
    if (s != FTP_OK) return s;
    float* own = dst->grad;
    dst->grad = grads->grad;                               // the update reads the gradients the other model's backward pass left
    s = sgd_range(dst, a, b, lr, nullptr, nullptr, (cudaStream_t)stream);
    dst->grad = own;
    return s;
}

extern "C" ftp_status ftp_aggregate_weights(ftp_model* dst, const ftp_model* const* srcs, int32_t n_src, int32_t a, int32_t b, void* stream) {
    FTP_REQUIRE(dst && srcs, FTP_EINVAL, "aggregate_weights: null argument");
    FTP_REQUIRE(n_src >= 1 && n_src <= 8, FTP_ERANGE, "aggregate_weights: 1 to 8 versions can be aggregated, not %d", n_src);
    ftp_status s = check_range(dst, a, b, "aggregate_weights");
    for (int k = 0; k < n_src && s == FTP_OK; ++k) s = same_architecture(dst, srcs[k], "aggregate_weights");
    if (s != FTP_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    for (int u = a; u < b; ++u) {
        const Arena& to = dst->arena[dst->owner[u]];
        MeanSources w{}, r{};
        w.n = r.n = n_src;
        for (int k = 0; k < n_src; ++k) {
            const Arena& from = srcs[k]->arena[srcs[k]->owner[u]];
            w.p[k] = from.w + dst->unit_p_off[u];
            r.p[k] = from.run + dst->unit_s_off[u];
        }
        Scope sc(dst, st, K_SGD, u, -1, 2, (double)(dst->unit_p_cnt[u] + dst->unit_s_cnt[u]) * 4.0 * (n_src + 1), (double)(dst->unit_p_cnt[u] + dst->unit_s_cnt[u]) * n_src, 2);
        mean_f32(w, to.w + dst->unit_p_off[u], dst->unit_p_cnt[u], st);
        mean_f32(r, to.run + dst->unit_s_off[u], dst->unit_s_cnt[u], st);
    }
    refresh_derived(dst, a, b, st);
    return check_launches("aggregate_weights");
}

extern "C" ftp_status ftp_get_partition(const ftp_model* m, int32_t* points, int32_t* n_stages) {
    FTP_REQUIRE(m && points && n_stages, FTP_EINVAL, "get_partition: null argument");
    for (int i = 0; i <= m->n_stages; ++i) points[i] = m->points[i];
    *n_stages = m->n_stages;
    return FTP_OK;
}

extern "C" ftp_status ftp_recover(ftp_model* m, const ftp_failed_stage* failed, int32_t n_failed, const void* central, size_t central_bytes,
                                  const int32_t* p_new, int32_t n_new, int32_t* counts, void* stream) {
    FTP_REQUIRE(m && failed && p_new, FTP_EINVAL, "recover: null argument");
    const int n_cur = m->n_stages, L = m->L;
    std::vector<int32_t> fl(std::max(n_failed, 0)), kind(L), index(L);
    for (int k = 0; k < n_failed; ++k) fl[k] = failed[k].stage;
    ftp_status s = ftp_recovery_plan(m->points.data(), n_cur, fl.data(), n_failed, p_new, n_new, kind.data(), index.data());
    if (s != FTP_OK) return s;
    FTP_REQUIRE(p_new[n_new] == L, FTP_EINVAL, "recover: the new partition must end at unit %d", L);
    // survivors in order: new stage j is the worker that was stage alive[j] and keeps its arena
    std::vector<int> alive, worker;
    for (int i = 0; i < n_cur; ++i)
        if (std::find(fl.begin(), fl.end(), i) == fl.end()) { alive.push_back(i); worker.push_back(m->worker[i]); }
    auto unit_bytes = [&](int u) { return (size_t)(m->unit_p_cnt[u] + m->unit_s_cnt[u]) * 4; };
    size_t all_bytes = 0;
    std::vector<size_t> central_off(L);
    for (int u = 0; u < L; ++u) { central_off[u] = all_bytes; all_bytes += unit_bytes(u); }
    // where each failed stage's units lie inside its chain replica; all checks before the first copy
    std::vector<const ftp_failed_stage*> rec(n_cur, nullptr);
    for (int k = 0; k < n_failed; ++k) {
        const ftp_failed_stage& f = failed[k];
        rec[f.stage] = &f;
        if (!f.replica) continue;
        size_t need = 0;
        for (int u = m->points[f.stage]; u < m->points[f.stage + 1]; ++u) need += unit_bytes(u);
        FTP_REQUIRE(f.replica_bytes == need, FTP_ESTATE, "recover: the replica of stage %d has %zu bytes, the stage's units take %zu (was it taken under another partition?)",
                    f.stage, f.replica_bytes, need);
    }
    for (int u = 0; u < L; ++u) {
        if (kind[u] != FTP_SRC_REPLICA && kind[u] != FTP_SRC_CENTRAL) continue;
        int holder = 0;
        while (!(m->points[holder] <= u && u < m->points[holder + 1])) ++holder;
        if (kind[u] == FTP_SRC_REPLICA && !rec[holder]->replica) kind[u] = FTP_SRC_CENTRAL;        // no chain replica was ever taken
        if (kind[u] == FTP_SRC_CENTRAL)
            FTP_REQUIRE(central && central_bytes >= all_bytes, FTP_ESTATE, "recover: unit %d is lost (no chain replica survives and the global replica is %s)", u,
                        central ? "too short" : "missing");
    }
    cudaStream_t st = (cudaStream_t)stream;
    int n_stage = 0, n_replica = 0, n_central = 0;
    std::vector<int> reloaded;
    for (int j = 0; j < n_new; ++j)
        for (int u = p_new[j]; u < p_new[j + 1]; ++u) {
            if (kind[u] == FTP_SRC_LOCAL) continue;
            Scope sc(m, st, K_COPY, u, -1, 2, 2.0 * unit_bytes(u), 0.0, 0);
            if (kind[u] == FTP_SRC_STAGE) {
                ++n_stage;
                s = copy_unit(m, u, worker[index[u]], worker[j], st);
                if (s != FTP_OK) return s;
                continue;
            }
            // from a replica: weights and running statistics as they were replicated; momentum restarts
            const char* src;
            cudaMemcpyKind how;
            if (kind[u] == FTP_SRC_REPLICA) {
                int holder = 0;
                while (!(m->points[holder] <= u && u < m->points[holder + 1])) ++holder;
                size_t off = 0;
                for (int v = m->points[holder]; v < u; ++v) off += unit_bytes(v);
                src = (const char*)rec[holder]->replica + off;
                how = rec[holder]->replica_is_host ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice;
                ++n_replica;
            } else {
                src = (const char*)central + central_off[u];
                how = cudaMemcpyHostToDevice;
                ++n_central;
            }
            const Arena& to = m->arena[worker[j]];
            if (m->unit_p_cnt[u]) CUDA_OK(cudaMemcpyAsync(to.w + m->unit_p_off[u], src, (size_t)m->unit_p_cnt[u] * 4, how, st));
            if (m->unit_s_cnt[u]) CUDA_OK(cudaMemcpyAsync(to.run + m->unit_s_off[u], src + (size_t)m->unit_p_cnt[u] * 4, (size_t)m->unit_s_cnt[u] * 4, how, st));
            reloaded.push_back(u);
        }
    // commit: the survivors' list and the owner table switch, then the derived copies of the reloaded weights are rebuilt
    for (int j = 0; j < n_new; ++j)
        for (int u = p_new[j]; u < p_new[j + 1]; ++u) m->owner[u] = worker[j];
    m->worker = worker;
    m->points.assign(p_new, p_new + n_new + 1);
    m->n_stages = n_new;
    std::fill(m->fwd_done.begin(), m->fwd_done.end(), 0);
    for (int u : reloaded) {
        const Arena& ar = m->arena[m->owner[u]];
        const long long po = m->unit_p_off[u], pc = m->unit_p_cnt[u];
        m->mom_init[u] = 0;
        if (!pc) continue;
        if (ar.wb) { f32_to_bf16(ar.w + po, ar.wb + po, pc, st); refresh_transposed(m, u, u + 1, st); }
        if (ar.wl) { tf32_lo(ar.w + po, ar.wl + po, pc, st); refresh_transposed(m, u, u + 1, st); }
    }
    if (counts) { counts[0] = n_stage; counts[1] = n_replica; counts[2] = n_central; }
    return check_launches("recover");
}

extern "C" ftp_status ftp_snapshot_weights(const ftp_model* m, int32_t stage, void* dst, size_t dst_bytes, int32_t dst_is_host, size_t* written,
                                           void* stream) {
    FTP_REQUIRE(m && dst, FTP_EINVAL, "snapshot_weights: null argument");
    FTP_REQUIRE(stage >= 0 && stage < m->n_stages, FTP_ERANGE, "snapshot_weights: stage %d out of range (%d stages)", stage, m->n_stages);
    const int a = m->points[stage], b = m->points[stage + 1];
    size_t need = 0;
    for (int u = a; u < b; ++u) need += (size_t)(m->unit_p_cnt[u] + m->unit_s_cnt[u]) * 4;
    FTP_REQUIRE(need <= dst_bytes, FTP_ERANGE, "snapshot_weights: stage %d needs %zu bytes, buffer has %zu", stage, need, dst_bytes);
    cudaStream_t st = (cudaStream_t)stream;
    const cudaMemcpyKind kind = dst_is_host ? cudaMemcpyDeviceToHost : cudaMemcpyDeviceToDevice;
    char* p = (char*)dst;
    const Arena& ar = m->arena[m->worker[stage]];
    Scope sc(const_cast<ftp_model*>(m), st, K_COPY, a, -1, 2, 2.0 * need, 0.0, 0);
    for (int u = a; u < b; ++u) {
        if (m->unit_p_cnt[u]) { CUDA_OK(cudaMemcpyAsync(p, ar.w + m->unit_p_off[u], (size_t)m->unit_p_cnt[u] * 4, kind, st)); p += m->unit_p_cnt[u] * 4; }
        if (m->unit_s_cnt[u]) { CUDA_OK(cudaMemcpyAsync(p, ar.run + m->unit_s_off[u], (size_t)m->unit_s_cnt[u] * 4, kind, st)); p += m->unit_s_cnt[u] * 4; }
    }
    if (written) *written = need;
    return FTP_OK;
}

extern "C" ftp_status ftp_trace_enable(ftp_model* m, int32_t on) {
    FTP_REQUIRE(m, FTP_EINVAL, "trace_enable: null model");
    m->trace = on != 0;
    return FTP_OK;
}

extern "C" ftp_status ftp_trace_read(ftp_model* m, ftp_trace_rec* out, int32_t max, int32_t* total) {
    FTP_REQUIRE(m && total && (out || max == 0), FTP_EINVAL, "trace_read: null argument");
    CUDA_OK(cudaDeviceSynchronize());
    *total = (int32_t)m->tr_used;
    for (size_t i = 0; i < m->tr_used; ++i) {
        float ms = 0.f;
        cudaEventElapsedTime(&ms, m->tr[i].e0, m->tr[i].e1);
        m->tr[i].rec.ms = ms;
        if ((int32_t)i < max) out[i] = m->tr[i].rec;
    }
    m->tr_used = 0;
    return FTP_OK;
}

#ifdef FTP_TIMELINE
namespace ftp {
static std::vector<void (*)(std::vector<unsigned long long>&, bool)>& tl_readers() {
    static std::vector<void (*)(std::vector<unsigned long long>&, bool)> v;
    return v;
}
void tl_register(void (*reader)(std::vector<unsigned long long>&, bool)) { tl_readers().push_back(reader); }
struct TlLaunch { const void* kernel; unsigned long long signature; const void* stream; };
static std::vector<TlLaunch> g_tl_launched;
void tl_note_launch(const void* kernel, unsigned long long signature, const void* stream) {
    if (g_tl_launched.size() < (1u << 20)) g_tl_launched.push_back({kernel, signature, stream});
}
}  // namespace ftp
// Measurement build only: the kernels launched since the last reset, one per line in launch order: mangled name, tab,
// signature of the grid (decimal), tab, stream (hex).
extern "C" int32_t ftp_debug_launch_names(char* buf, int32_t cap, int32_t reset) {
    size_t used = 0;
    int32_t n = 0;
    for (const ftp::TlLaunch& l : ftp::g_tl_launched) {
        const char* fn = nullptr;
        if (cudaFuncGetName(&fn, l.kernel) != cudaSuccess || !fn) fn = "?";
        char tail[64];
        std::snprintf(tail, sizeof tail, "\t%llu\t%p", l.signature, l.stream);
        const std::string line = std::string(fn) + tail;
        const char* name = line.c_str();
        const size_t len = line.size();
        if (used + len + 2 > (size_t)std::max(cap, 0)) break;
        std::memcpy(buf + used, name, len);
        used += len;
        buf[used++] = '\n';
        ++n;
    }
    if (cap > 0) buf[used < (size_t)cap ? used : (size_t)cap - 1] = 0;
    if (reset) ftp::g_tl_launched.clear();
    return n;
}
// Measurement build only: the start time (ns of the global timer) and the signature of every grid launched since the last
// reset, merged over the translation units and sorted by time: out[2 i] = time, out[2 i + 1] = signature, at most `max`
// entries; returns the number of entries there are; synchronises the device.
extern "C" int32_t ftp_debug_timeline(unsigned long long* out, int32_t max, int32_t reset) {
    cudaDeviceSynchronize();
    std::vector<unsigned long long> raw;
    for (auto r : ftp::tl_readers()) r(raw, reset != 0);
    std::vector<std::pair<unsigned long long, unsigned long long>> all(raw.size() / 2);
    for (size_t i = 0; i < all.size(); ++i) all[i] = {raw[2 * i], raw[2 * i + 1]};
    std::sort(all.begin(), all.end());
    const int32_t n = (int32_t)std::min<size_t>(all.size(), (size_t)std::max(max, 0));
    for (int32_t i = 0; i < n; ++i) { out[2 * i] = all[i].first; out[2 * i + 1] = all[i].second; }
    return (int32_t)all.size();
}
#endif

extern "C" const char* ftp_kernel_name(int32_t kernel) { return kernel >= 0 && kernel < K_COUNT ? kKernelNames[kernel] : "?"; }

extern "C" ftp_status ftp_launch_count(const ftp_model* m, int64_t* launches) {
    FTP_REQUIRE(m && launches, FTP_EINVAL, "launch_count: null argument");
    *launches = g_launches;
    return FTP_OK;
}
