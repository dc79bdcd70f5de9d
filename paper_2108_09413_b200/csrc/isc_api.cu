// Host side of libisc: argument checks, model repacking and upload, launch sequencing of the
// Monte-Carlo loop (Algorithm 1 steps 1-4, Algorithm 2 steps 1-2) and the decision rules.
#include <cuda_runtime.h>

#include <chrono>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <new>
#include <thread>
#include <vector>

#include "isc.h"
#include "isc_internal.h"
#include "isc_line.h"

using namespace isc;

namespace {

inline int pad16(int c) { return (c + 15) & ~15; }

struct HostLayer {           // private copy of one isc_layer with its arrays
    isc_layer d;
    std::vector<int8_t> w;
    std::vector<int32_t> bias, mult;
    std::vector<int8_t> shift;
};

struct DevBuf {
    void *p = nullptr;
    size_t bytes = 0;
};

}  // namespace

struct isc_model {
    int in_c = 0, in_h = 0, in_w = 0, n_classes = 0;
    std::vector<HostLayer> layers;
    std::vector<TShape> shapes;                 // [n_layers + 1]
    int64_t macs = 0;

    // device parameters of the layer-by-layer engine
    std::vector<GLayer> glayers;
    std::vector<void *> param_allocs;
    std::vector<const int8_t *> wpacks;         // per layer: repacked weights of the tensor-core convolution, or null
    std::vector<const int32_t *> tc_cst;        // per layer: its epilogue constants
    std::vector<char> tc_fast;
    std::vector<uint32_t> tc_resk;           // per layer: offset of the residual term's two-instruction form, or 0xFFFFFFFF
    bool has_tc = false;
    int32_t *d_tc_err = nullptr;

    // activation buffers: tensor t lives in pool buffer tensor_buf[t] (bytes per sample buf_bytes[b])
    std::vector<int> tensor_buf;
    std::vector<size_t> buf_bytes;
    std::vector<DevBuf> bufs;
    int ws_batch = 0;

    // per-call device scratch
    uint8_t *d_x = nullptr;       size_t d_x_bytes = 0;
    int32_t *d_counts = nullptr;  size_t d_counts_n = 0;
    int8_t *d_logits = nullptr;   size_t d_logits_bytes = 0;
    uint32_t *d_cum = nullptr;    size_t d_cum_n = 0;
    double cum_sigma = -1.0;
    int cum_T = 0, cum_kind = -1, cum_steps = 0;

    isc::LinePlan *line = nullptr;

    // isc_certify_batch: pinned copy of the vote counts, one event per image
    int32_t *h_counts = nullptr;  size_t h_counts_bytes = 0;
    std::vector<cudaEvent_t> events;

    int64_t opt_batch = 0, opt_engine = 0, opt_noise = 0, opt_tensor_copy = 1;
    int64_t last_engine = 0, launches = 0;
};

namespace {

#define CK(call)                                      \
    do {                                              \
        cudaError_t e_ = (call);                      \
        if (e_ != cudaSuccess) {                      \
            if (getenv("ISC_DEBUG_CUDA")) fprintf(stderr, "isc: %s: %s\n", #call, cudaGetErrorString(e_)); \
            cudaGetLastError();                       \
            return e_ == cudaErrorMemoryAllocation ? ISC_ERR_NOMEM : ISC_ERR_CUDA; \
        }                                             \
    } while (0)

int infer_shape(const isc_layer &L, const TShape &in, TShape *out)
{
    switch (L.op) {
    case ISC_CONV2D:
    case ISC_MAXPOOL:
        if (L.kh < 1 || L.kw < 1 || L.stride < 1 || L.pad < 0) return ISC_ERR_SHAPE;
        if (L.cin != in.c) return ISC_ERR_SHAPE;
        if (in.h + 2 * L.pad < L.kh || in.w + 2 * L.pad < L.kw) return ISC_ERR_SHAPE;
        if (L.op == ISC_MAXPOOL && L.cout != L.cin) return ISC_ERR_SHAPE;
        if (L.cout < 1) return ISC_ERR_SHAPE;
        out->c = L.cout;
        out->h = (in.h + 2 * L.pad - L.kh) / L.stride + 1;
        out->w = (in.w + 2 * L.pad - L.kw) / L.stride + 1;
        break;
    case ISC_FC:
        if (in.h != 1 || in.w != 1 || L.cin != in.c || L.cout < 1) return ISC_ERR_SHAPE;
        out->c = L.cout; out->h = 1; out->w = 1;
        break;
    case ISC_GAVGPOOL:
        if (L.cin != in.c || L.cout != in.c) return ISC_ERR_SHAPE;
        out->c = in.c; out->h = 1; out->w = 1;
        break;
    default:
        return ISC_ERR_ARG;
    }
    out->cp = pad16(out->c);
    return ISC_OK;
}

template <typename T>
int upload(isc_model *m, const std::vector<T> &h, const T **dptr)
{
    void *p = nullptr;
    CK(cudaMalloc(&p, std::max<size_t>(h.size() * sizeof(T), 16)));
    m->param_allocs.push_back(p);
    CK(cudaMemcpy(p, h.data(), h.size() * sizeof(T), cudaMemcpyHostToDevice));
    *dptr = static_cast<const T *>(p);
    return ISC_OK;
}

// Validate, copy, infer shapes.  No device work.
int build_host_model(isc_model *m, const isc_layer *layers, int n_layers)
{
    m->shapes.resize((size_t)n_layers + 1);
    m->shapes[0] = TShape{m->in_c, m->in_h, m->in_w, 4};
    m->layers.resize((size_t)n_layers);
    std::vector<int> uses_of_input(1, 0);
    for (int i = 0; i < n_layers; ++i) {
        const isc_layer &L = layers[i];
        if (L.op < ISC_CONV2D || L.op > ISC_MAXPOOL) return ISC_ERR_ARG;
        if (L.in_tensor < 0 || L.in_tensor > i) return ISC_ERR_SHAPE;
        if (L.res_tensor < -1 || L.res_tensor > i) return ISC_ERR_SHAPE;
        const bool weighted = L.op == ISC_CONV2D || L.op == ISC_FC;
        if (L.res_tensor >= 0 && !weighted) return ISC_ERR_SHAPE;
        if (!L.mult || !L.shift) return ISC_ERR_ARG;
        if (weighted && (!L.w || !L.bias)) return ISC_ERR_ARG;
        int rc = infer_shape(L, m->shapes[(size_t)L.in_tensor], &m->shapes[(size_t)i + 1]);
        if (rc) return rc;
        const TShape &os = m->shapes[(size_t)i + 1];
        if (L.res_tensor >= 0) {
            const TShape &r = m->shapes[(size_t)L.res_tensor];
            if (L.res_tensor == 0 || r.c != os.c || r.h != os.h || r.w != os.w) return ISC_ERR_SHAPE;
            if (L.res_mult < (1 << 30) || L.res_shift < -4 || L.res_shift > 4) return ISC_ERR_ARG;
            if (L.zp_res < -128 || L.zp_res > 127) return ISC_ERR_ARG;
        }
        const int zp_in_lo = L.in_tensor == 0 ? 0 : -128, zp_in_hi = L.in_tensor == 0 ? 255 : 127;
        if (L.zp_in < zp_in_lo || L.zp_in > zp_in_hi) return ISC_ERR_ARG;
        if (L.zp_out < -128 || L.zp_out > 127) return ISC_ERR_ARG;
        if (L.relu != 0 && L.relu != 1) return ISC_ERR_ARG;

        HostLayer &H = m->layers[(size_t)i];
        H.d = L;
        const int nch = weighted ? L.cout : 1;
        H.mult.assign(L.mult, L.mult + nch);
        H.shift.assign(L.shift, L.shift + nch);
        for (int c = 0; c < nch; ++c) {
            if (L.op != ISC_MAXPOOL && H.mult[(size_t)c] < (1 << 30)) return ISC_ERR_ARG;
            if (H.shift[(size_t)c] < 0 || H.shift[(size_t)c] > 31) return ISC_ERR_ARG;
        }
        if (weighted) {
            const int kh = L.op == ISC_FC ? 1 : L.kh, kw = L.op == ISC_FC ? 1 : L.kw;
            const size_t per_out = (size_t)L.cin * kh * kw;
            H.w.assign(L.w, L.w + per_out * L.cout);
            H.bias.assign(L.bias, L.bias + L.cout);
            H.d.kh = kh; H.d.kw = kw;
            if (L.op == ISC_FC) { H.d.stride = 1; H.d.pad = 0; }
            // worst-case accumulator magnitude must stay inside int32
            const int amax = 255;                              // |a - zp_in| <= 255 for 8-bit activations
            for (int o = 0; o < L.cout; ++o) {
                int64_t s = 0;
                for (size_t k = 0; k < per_out; ++k) {
                    const int wv = H.w[(size_t)o * per_out + k];
                    if (wv == -128) return ISC_ERR_ARG;        // symmetric int8 weights: [-127, 127]
                    s += std::abs(wv);
                }
                const int64_t b = H.bias[(size_t)o];
                if (s * amax + (b < 0 ? -b : b) >= (1ll << 30)) return ISC_ERR_UNSUPPORTED;
            }
            m->macs += (int64_t)os.h * os.w * L.cout * (int64_t)per_out;
        }
        H.d.w = nullptr; H.d.bias = nullptr; H.d.mult = nullptr; H.d.shift = nullptr;
    }
    const TShape &last = m->shapes[(size_t)n_layers];
    if (last.c != m->n_classes || last.h != 1 || last.w != 1) return ISC_ERR_SHAPE;
    return ISC_OK;
}

// Device parameters and buffer plan of the layer-by-layer engine.
int build_generic_engine(isc_model *m)
{
    const int n = (int)m->layers.size();
    // tensor 0 exists only inside the first convolution's staging
    const isc_layer &L0 = m->layers[0].d;
    if (L0.op != ISC_CONV2D || L0.in_tensor != 0 || L0.cin > 4) return ISC_ERR_UNSUPPORTED;
    for (int i = 1; i < n; ++i)
        if (m->layers[(size_t)i].d.in_tensor == 0) return ISC_ERR_UNSUPPORTED;

    m->glayers.resize((size_t)n);
    m->wpacks.assign((size_t)n, nullptr);
    m->tc_cst.assign((size_t)n, nullptr);
    m->tc_fast.assign((size_t)n, 0);
    m->tc_resk.assign((size_t)n, 0xFFFFFFFFu);
    for (int i = 0; i < n; ++i) {
        const HostLayer &H = m->layers[(size_t)i];
        const isc_layer &L = H.d;
        const TShape &is = m->shapes[(size_t)L.in_tensor], &os = m->shapes[(size_t)i + 1];
        GLayer G;
        memset(&G, 0, sizeof(G));
        G.op = L.op;
        G.cin = L.cin; G.cinp = i == 0 ? 4 : is.cp;
        G.cout = L.cout; G.coutp = os.cp;
        G.kh = L.kh; G.kw = L.kw; G.stride = L.stride; G.pad = L.pad; G.relu = L.relu;
        G.zp_in = L.zp_in; G.zp_out = L.zp_out; G.zp_res = L.zp_res;
        G.res_mult = L.res_mult; G.res_shift = L.res_shift;
        G.hin = is.h; G.win = is.w; G.hout = os.h; G.wout = os.w;
        const bool weighted = L.op == ISC_CONV2D || L.op == ISC_FC;
        std::vector<int32_t> mult((size_t)(weighted ? G.coutp : 1), 1 << 30), shift(mult.size(), 0);
        for (size_t c = 0; c < H.mult.size(); ++c) { mult[c] = H.mult[c]; shift[c] = H.shift[c]; }
        int rc = upload(m, mult, &G.mult); if (rc) return rc;
        rc = upload(m, shift, &G.shift); if (rc) return rc;
        if (weighted) {
            const int taps = L.kh * L.kw;
            std::vector<int32_t> bias((size_t)G.coutp, 0);
            for (int o = 0; o < L.cout; ++o) {
                int64_t s = 0;
                for (int k = 0; k < L.cin * taps; ++k) s += H.w[(size_t)o * L.cin * taps + k];
                bias[(size_t)o] = (int32_t)(H.bias[(size_t)o] - (int64_t)L.zp_in * s);   // padding value is zp_in
            }
            rc = upload(m, bias, &G.bias); if (rc) return rc;
            std::vector<int8_t> w;
            if (i == 0) {                                   // [coutp][taps][4]
                w.assign((size_t)G.coutp * taps * 4, 0);
                for (int o = 0; o < L.cout; ++o)
                    for (int c = 0; c < L.cin; ++c)
                        for (int t = 0; t < taps; ++t)
                            w[((size_t)o * taps + t) * 4 + c] = H.w[((size_t)o * L.cin + c) * taps + t];
            } else {                                        // [coutp/16][taps][cinp/16][16 out][16 in]
                const int c16s = G.cinp / 16;
                w.assign((size_t)G.coutp * taps * G.cinp, 0);
                for (int o = 0; o < L.cout; ++o)
                    for (int c = 0; c < L.cin; ++c)
                        for (int t = 0; t < taps; ++t) {
                            const size_t idx = ((((size_t)(o / 16) * taps + t) * c16s + c / 16) * 16 + o % 16) * 16 + c % 16;
                            w[idx] = H.w[((size_t)o * L.cin + c) * taps + t];
                        }
            }
            rc = upload(m, w, &G.w); if (rc) return rc;
            if (i == 0 && stem_fits(G, m->in_c)) {          // the stem for the tensor-core kernel
                std::vector<int8_t> wp(stem_pack_bytes(G));
                stem_pack_weights(G, H.w.data(), wp.data());
                rc = upload(m, wp, &m->wpacks[0]); if (rc) return rc;
                std::vector<int32_t> c4((size_t)G.coutp * 4);
                m->tc_fast[0] = igemm_constants(G, bias.data(), mult.data(), shift.data(), c4.data(), false, nullptr) ? 1 : 0;
                rc = upload(m, c4, &m->tc_cst[0]); if (rc) return rc;
            }
            if (i > 0 && igemm_tile_n(G)) {                 // the same layer for the tensor-core kernel
                std::vector<int8_t> wp(igemm_pack_bytes(G));
                igemm_pack_weights(G, H.w.data(), wp.data());
                rc = upload(m, wp, &m->wpacks[(size_t)i]); if (rc) return rc;
                std::vector<int32_t> c4((size_t)G.coutp * 4);
                m->tc_fast[(size_t)i] = igemm_constants(G, bias.data(), mult.data(), shift.data(), c4.data(), H.d.res_tensor >= 0, &m->tc_resk[(size_t)i]) ? 1 : 0;
                rc = upload(m, c4, &m->tc_cst[(size_t)i]); if (rc) return rc;
                m->has_tc = true;
            }
        }
        m->glayers[(size_t)i] = G;
    }
    if (m->has_tc) {
        std::vector<int32_t> zero(1, 0);
        const int32_t *p = nullptr;
        int rc = upload(m, zero, &p); if (rc) return rc;
        m->d_tc_err = const_cast<int32_t *>(p);
    }

    // buffer plan: greedy reuse by last use
    std::vector<int> last_use((size_t)n + 1, -1);
    for (int i = 0; i < n; ++i) {
        last_use[(size_t)m->layers[(size_t)i].d.in_tensor] = i;
        if (m->layers[(size_t)i].d.res_tensor >= 0) last_use[(size_t)m->layers[(size_t)i].d.res_tensor] = i;
    }
    last_use[(size_t)n] = n;
    m->tensor_buf.assign((size_t)n + 1, -1);
    std::vector<int> owner;                                 // pool buffer -> tensor currently in it (or -1)
    for (int i = 0; i < n; ++i) {
        const int t = i + 1;
        const TShape &s = m->shapes[(size_t)t];
        const size_t need = (size_t)s.h * s.w * s.cp;
        for (size_t b = 0; b < owner.size(); ++b)           // release buffers whose tensor is dead
            if (owner[b] >= 0 && last_use[(size_t)owner[b]] < i) owner[b] = -1;
        int pick = -1;
        for (size_t b = 0; b < owner.size(); ++b)
            if (owner[b] < 0 && (pick < 0 || m->buf_bytes[b] > m->buf_bytes[(size_t)pick])) pick = (int)b;
        if (pick < 0) {
            owner.push_back(-1);
            m->buf_bytes.push_back(0);
            pick = (int)owner.size() - 1;
        }
        m->buf_bytes[(size_t)pick] = std::max(m->buf_bytes[(size_t)pick], need);
        owner[(size_t)pick] = t;
        m->tensor_buf[(size_t)t] = pick;
    }
    m->bufs.resize(owner.size());
    return ISC_OK;
}

int ensure_bytes(void **p, size_t *have, size_t need)
{
    if (*have >= need && *p) return ISC_OK;
    if (*p) cudaFree(*p);
    *p = nullptr; *have = 0;
    CK(cudaMalloc(p, std::max<size_t>(need, 16)));
    *have = need;
    return ISC_OK;
}

int ensure_workspace(isc_model *m, int batch)
{
    if (batch <= m->ws_batch) return ISC_OK;
    for (size_t b = 0; b < m->bufs.size(); ++b) {
        if (m->bufs[b].p) cudaFree(m->bufs[b].p);
        m->bufs[b].p = nullptr;
    }
    m->ws_batch = 0;
    for (size_t b = 0; b < m->bufs.size(); ++b) {
        CK(cudaMalloc(&m->bufs[b].p, m->buf_bytes[b] * (size_t)batch));
        m->bufs[b].bytes = m->buf_bytes[b] * (size_t)batch;
    }
    m->ws_batch = batch;
    return ISC_OK;
}

int ensure_noise_table(isc_model *m, double sigma, cudaStream_t st)
{
    if (m->d_cum && m->cum_sigma == sigma && m->cum_kind == (int)m->opt_noise) return ISC_OK;
    std::vector<uint32_t> cum;
    if (m->opt_noise) noise_table_rounded(sigma, cum); else noise_table(sigma, cum);
    // the guide table follows the cumulative one in the same allocation
    const size_t n_cum = cum.size();
    for (int j = 0; j <= isc::kNoiseGuide; ++j) {
        const uint64_t u = (uint64_t)j << (32 - isc::kNoiseGuideBits);
        uint32_t i = 0;
        while (i + 1 < n_cum && u >= cum[i]) ++i;        // min{ i : u < cum[i] }, the last entry matching always
        cum.push_back(i);
    }
    size_t have = m->d_cum_n * sizeof(uint32_t);
    void *p = m->d_cum;
    int rc = ensure_bytes(&p, &have, cum.size() * sizeof(uint32_t));
    m->d_cum = (uint32_t *)p; m->d_cum_n = have / sizeof(uint32_t);
    if (rc) return rc;
    CK(cudaMemcpyAsync(m->d_cum, cum.data(), cum.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, st));
    CK(cudaStreamSynchronize(st));                       // cum is a local vector
    m->cum_sigma = sigma;
    m->cum_kind = (int)m->opt_noise;
    m->cum_T = (int)(n_cum - 1) / 2;
    // bisection steps that close the widest guide interval
    uint32_t span = 0;
    for (int j = 0; j < isc::kNoiseGuide; ++j) span = std::max(span, cum[n_cum + j + 1] - cum[n_cum + j]);
    m->cum_steps = 0;
    while ((1u << m->cum_steps) < span + 1) ++m->cum_steps;
    return ISC_OK;
}

int check_stream_args(uint64_t image_id, int32_t phase, int64_t first, int64_t n, double sigma)
{
    if (!(sigma > 0.0) || !std::isfinite(sigma) || sigma > 64.0) return ISC_ERR_ARG;
    if (phase < 0 || phase > 255) return ISC_ERR_ARG;
    if (image_id >= (1ull << 48)) return ISC_ERR_ARG;
    if (first < 0 || n < 0 || first + n > (1ll << 40)) return ISC_ERR_ARG;
    return ISC_OK;
}

NoiseStream make_stream(const isc_model *m, uint64_t seed, uint64_t image_id, int32_t phase, int64_t first)
{
    NoiseStream ns;
    ns.key0 = (uint32_t)(seed & 0xFFFFFFFFu);
    ns.key1 = (uint32_t)(seed >> 32);
    ns.ctr2 = (uint32_t)(image_id & 0xFFFFFFFFu);
    ns.ctr3_fixed = (uint32_t)phase | (uint32_t)(((image_id >> 32) & 0xFFFFu) << 16);
    ns.first_sample = first;
    ns.cum = m->d_cum;
    ns.T = m->cum_T;
    ns.guide = m->d_cum ? m->d_cum + (2 * m->cum_T + 1) : nullptr;
    ns.guide_steps = m->cum_steps;
    return ns;
}

int choose_engine(isc_model *m)
{
    if (m->opt_engine == 1) return 1;
    if (m->opt_engine == 2) return m->has_tc ? 2 : ISC_ERR_UNSUPPORTED;
    if (m->opt_engine == 3) return m->line ? 3 : ISC_ERR_UNSUPPORTED;
    if (m->line) return 3;
    if (m->has_tc) return 2;
    return 1;
}

// Layer-by-layer forward of `batch` samples; leaves the logits in the last tensor's buffer.
int generic_forward(isc_model *m, const uint8_t *d_x, const NoiseStream &ns, int batch, cudaStream_t st,
                    int stop_after_layer = -1, bool tensor_cores = false)
{
    const int n = (int)m->glayers.size();
    for (int i = 0; i < n; ++i) {
        const GLayer &G = m->glayers[(size_t)i];
        const isc_layer &L = m->layers[(size_t)i].d;
        int8_t *out = (int8_t *)m->bufs[(size_t)m->tensor_buf[(size_t)i + 1]].p;
        const int8_t *in = i == 0 ? nullptr : (const int8_t *)m->bufs[(size_t)m->tensor_buf[(size_t)L.in_tensor]].p;
        const int8_t *res = L.res_tensor >= 0 ? (const int8_t *)m->bufs[(size_t)m->tensor_buf[(size_t)L.res_tensor]].p : nullptr;
        cudaError_t e;
        if (i == 0 && tensor_cores && m->wpacks[0])
            e = launch_stem_conv(G, m->wpacks[0], m->tc_cst[0], m->tc_fast[0] != 0, d_x, m->in_c, ns, batch, out, m->d_tc_err, st);
        else if (i == 0) e = launch_first_conv(G, d_x, m->in_c, ns, batch, out, st);
        else if (tensor_cores && m->wpacks[(size_t)i]) e = launch_igemm_conv(G, m->wpacks[(size_t)i], m->tc_cst[(size_t)i], m->tc_fast[(size_t)i] != 0, m->tc_resk[(size_t)i], batch, in, res, out, m->d_tc_err, st, false, m->opt_tensor_copy != 0);
        else if (L.op == ISC_CONV2D || L.op == ISC_FC) e = launch_conv(G, batch, in, res, out, st);
        else if (L.op == ISC_GAVGPOOL) e = launch_gavgpool(G, batch, in, out, st);
        else e = launch_maxpool(G, batch, in, out, st);
        m->launches += 1;
        if (e != cudaSuccess) {
            if (getenv("ISC_DEBUG_CUDA")) fprintf(stderr, "isc: layer %d launch: %s\n", i, cudaGetErrorString(e));
            return ISC_ERR_CUDA;
        }
        if (i == stop_after_layer) break;
    }
    return ISC_OK;
}

size_t generic_bytes_per_sample(const isc_model *m)
{
    size_t s = 0;
    for (size_t b : m->buf_bytes) s += b;
    return s;
}

// The Monte-Carlo loop for one image and one phase; adds votes into d_counts (device).
int run_counts(isc_model *m, const uint8_t *d_x, uint64_t seed, uint64_t image_id, int32_t phase,
               int64_t first, int64_t n, cudaStream_t st, int32_t *d_counts, int8_t *d_logits)
{
    const int engine = choose_engine(m);
    if (engine < 0) return engine;
    m->last_engine = engine;
    if (engine == 3) {
        NoiseStream ns = make_stream(m, seed, image_id, phase, first);
        int64_t launches = 0;
        int rc = isc::line_run(m->line, d_x, ns, n, (int)m->opt_batch, d_counts, d_logits, st, &launches);
        m->launches += launches;
        return rc;
    }
    int64_t cap = m->opt_batch > 0 ? m->opt_batch : 4096;
    const size_t per = std::max<size_t>(generic_bytes_per_sample(m), 1);
    cap = std::min<int64_t>(cap, std::max<int64_t>(1, (int64_t)((3ull << 30) / per)));
    cap = std::min<int64_t>(cap, 32768);
    const int batch_alloc = (int)std::min<int64_t>(cap, std::max<int64_t>(n, 1));
    int rc = ensure_workspace(m, batch_alloc);
    if (rc) return rc;
    const int last = (int)m->glayers.size();
    for (int64_t done = 0; done < n; done += cap) {
        const int b = (int)std::min<int64_t>(cap, n - done);
        NoiseStream ns = make_stream(m, seed, image_id, phase, first + done);
        rc = generic_forward(m, d_x, ns, b, st, -1, engine == 2);
        if (rc) return rc;
        const int8_t *lg = (const int8_t *)m->bufs[(size_t)m->tensor_buf[(size_t)last]].p;
        cudaError_t e = launch_votes(lg, m->shapes[(size_t)last].cp, m->n_classes, b, d_counts,
                                     d_logits ? d_logits + (size_t)done * m->n_classes : nullptr, st);
        m->launches += 1;
        if (e != cudaSuccess) return ISC_ERR_CUDA;
    }
    return ISC_OK;
}

int stage_image(isc_model *m, const uint8_t *x, size_t bytes, bool on_device, cudaStream_t st,
                const uint8_t **d_x)
{
    if (on_device) { *d_x = x; return ISC_OK; }
    void *p = m->d_x; size_t have = m->d_x_bytes;
    int rc = ensure_bytes(&p, &have, bytes);
    m->d_x = (uint8_t *)p; m->d_x_bytes = have;
    if (rc) return rc;
    CK(cudaMemcpyAsync(m->d_x, x, bytes, cudaMemcpyHostToDevice, st));
    *d_x = m->d_x;
    return ISC_OK;
}

// After the stream has been synchronised: has a bounded wait of a tensor-core kernel expired?
int check_engines(isc_model *m)
{
    int rc;
    if (m->line && (rc = isc::line_check(m->line))) return rc;
    if (m->d_tc_err && m->last_engine == 2) {
        int32_t e = 0;
        CK(cudaMemcpy(&e, m->d_tc_err, sizeof(e), cudaMemcpyDeviceToHost));
        if (e != 0) {
            cudaMemset(m->d_tc_err, 0, sizeof(e));
            return ISC_ERR_TIMEOUT;
        }
    }
    return ISC_OK;
}

int ensure_counts(isc_model *m, size_t n)
{
    void *p = m->d_counts; size_t have = m->d_counts_n * sizeof(int32_t);
    int rc = ensure_bytes(&p, &have, n * sizeof(int32_t));
    m->d_counts = (int32_t *)p; m->d_counts_n = have / sizeof(int32_t);
    return rc;
}

}  // namespace

// =============================================================================== C ABI

extern "C" {

const char *isc_strerror(int code)
{
    switch (code) {
    case ISC_OK: return "ok";
    case ISC_ERR_ARG: return "invalid argument";
    case ISC_ERR_SHAPE: return "layer list does not type-check";
    case ISC_ERR_UNSUPPORTED: return "not supported by the kernels";
    case ISC_ERR_NOMEM: return "out of memory";
    case ISC_ERR_CUDA: return "CUDA error";
    case ISC_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown error";
    }
}

int isc_load_qmodel(const isc_layer *layers, int n_layers, int in_c, int in_h, int in_w, int n_classes,
                    isc_model **out)
{
    if (!layers || !out || n_layers < 1 || n_layers > 4096) return ISC_ERR_ARG;
    if (in_c < 1 || in_h < 1 || in_w < 1 || n_classes < 1 || n_classes > 4096) return ISC_ERR_ARG;
    if ((int64_t)in_c * in_h * in_w > (1ll << 30)) return ISC_ERR_ARG;
    isc_model *m = new (std::nothrow) isc_model();
    if (!m) return ISC_ERR_NOMEM;
    m->in_c = in_c; m->in_h = in_h; m->in_w = in_w; m->n_classes = n_classes;
    int rc;
    try {
        rc = build_host_model(m, layers, n_layers);
        if (rc == ISC_OK) rc = build_generic_engine(m);
        if (rc == ISC_OK) {
            std::vector<isc::LayerIn> ml(m->layers.size());
            for (size_t i = 0; i < m->layers.size(); ++i) {
                const HostLayer &H = m->layers[i];
                ml[i].d = H.d;
                ml[i].w = H.w.data(); ml[i].bias = H.bias.data();
                ml[i].mult = H.mult.data(); ml[i].shift = H.shift.data();
            }
            rc = isc::line_build(ml.data(), (int)ml.size(), in_c, in_h, in_w, n_classes, &m->line);
        }
    } catch (const std::bad_alloc &) {
        rc = ISC_ERR_NOMEM;
    }
    if (rc != ISC_OK) {
        isc_free_qmodel(m);
        return rc;
    }
    *out = m;
    return ISC_OK;
}

int isc_plan_resident(const isc_layer *layers, int n_layers, int in_c, int in_h, int in_w, int n_classes,
                      int32_t *out_rule, int64_t *out_smem_bytes)
{
    if (!layers || n_layers < 1 || n_layers > 4096) return ISC_ERR_ARG;
    if (in_c < 1 || in_h < 1 || in_w < 1 || n_classes < 1 || n_classes > 4096) return ISC_ERR_ARG;
    if ((int64_t)in_c * in_h * in_w > (1ll << 30)) return ISC_ERR_ARG;
    try {
        isc_model m;
        m.in_c = in_c; m.in_h = in_h; m.in_w = in_w; m.n_classes = n_classes;
        int rc = build_host_model(&m, layers, n_layers);
        if (rc) return rc;
        std::vector<isc::LayerIn> ml(m.layers.size());
        for (size_t i = 0; i < m.layers.size(); ++i) {
            const HostLayer &H = m.layers[i];
            ml[i].d = H.d;
            ml[i].w = H.w.data(); ml[i].bias = H.bias.data();
            ml[i].mult = H.mult.data(); ml[i].shift = H.shift.data();
        }
        int rule = 0;
        uint32_t smem = 0;
        const int fits = isc::line_plan_probe(ml.data(), (int)ml.size(), in_c, in_h, in_w, n_classes, &rule, &smem);
        if (out_rule) *out_rule = rule;
        if (out_smem_bytes) *out_smem_bytes = smem;
        return fits;
    } catch (const std::bad_alloc &) {
        return ISC_ERR_NOMEM;
    }
}

void isc_free_qmodel(isc_model *m)
{
    if (!m) return;
    for (void *p : m->param_allocs) cudaFree(p);
    for (DevBuf &b : m->bufs) if (b.p) cudaFree(b.p);
    if (m->d_x) cudaFree(m->d_x);
    if (m->d_counts) cudaFree(m->d_counts);
    if (m->d_logits) cudaFree(m->d_logits);
    if (m->d_cum) cudaFree(m->d_cum);
    if (m->h_counts) cudaFreeHost(m->h_counts);
    for (cudaEvent_t ev : m->events) cudaEventDestroy(ev);
    isc::line_free(m->line);
    delete m;
}

int isc_sample_counts(isc_model *m, const uint8_t *x_u8, uint64_t seed, uint64_t image_id, int32_t phase,
                      int64_t first_sample, int64_t n_samples, double sigma, void *cuda_stream,
                      int32_t *out_counts, int8_t *out_logits)
{
    if (!m || !x_u8 || !out_counts) return ISC_ERR_ARG;
    int rc = check_stream_args(image_id, phase, first_sample, n_samples, sigma);
    if (rc) return rc;
    if (n_samples > (1ll << 31) - 1) return ISC_ERR_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t C = (size_t)m->n_classes;
    if ((rc = ensure_noise_table(m, sigma, st))) return rc;
    if ((rc = ensure_counts(m, C))) return rc;
    const uint8_t *d_x;
    if ((rc = stage_image(m, x_u8, (size_t)m->in_c * m->in_h * m->in_w, false, st, &d_x))) return rc;
    if (out_logits) {
        void *p = m->d_logits; size_t have = m->d_logits_bytes;
        rc = ensure_bytes(&p, &have, (size_t)std::max<int64_t>(n_samples, 1) * C);
        m->d_logits = (int8_t *)p; m->d_logits_bytes = have;
        if (rc) return rc;
    }
    CK(cudaMemsetAsync(m->d_counts, 0, C * sizeof(int32_t), st));
    if ((rc = run_counts(m, d_x, seed, image_id, phase, first_sample, n_samples, st, m->d_counts,
                         out_logits ? m->d_logits : nullptr))) {
        cudaStreamSynchronize(st);
        return rc;
    }
    std::vector<int32_t> h(C);
    std::vector<int8_t> hl;
    CK(cudaMemcpyAsync(h.data(), m->d_counts, C * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    if (out_logits && n_samples > 0) {
        hl.resize((size_t)n_samples * C);
        CK(cudaMemcpyAsync(hl.data(), m->d_logits, hl.size(), cudaMemcpyDeviceToHost, st));
    }
    CK(cudaStreamSynchronize(st));
    if ((rc = check_engines(m))) return rc;
    memcpy(out_counts, h.data(), C * sizeof(int32_t));
    if (out_logits && n_samples > 0) memcpy(out_logits, hl.data(), hl.size());
    return ISC_OK;
}

int isc_predict(isc_model *m, const uint8_t *x_u8, uint64_t seed, uint64_t image_id, int64_t N, double sigma,
                double alpha, void *cuda_stream, int32_t *out_class, int32_t *out_counts)
{
    if (!m || !x_u8 || !out_class) return ISC_ERR_ARG;
    if (N < 1 || !(alpha > 0.0 && alpha < 1.0)) return ISC_ERR_ARG;
    std::vector<int32_t> counts((size_t)m->n_classes);
    int rc = isc_sample_counts(m, x_u8, seed, image_id, 2, 0, N, sigma, cuda_stream, counts.data(), nullptr);
    if (rc) return rc;
    *out_class = decide_predict(counts.data(), m->n_classes, alpha);
    if (out_counts) memcpy(out_counts, counts.data(), counts.size() * sizeof(int32_t));
    return ISC_OK;
}

int isc_certify_batch(isc_model *m, const uint8_t *x_u8, int x_on_device, int n_images, uint64_t seed,
                      uint64_t image_id0, int64_t N0, int64_t N, double sigma, double alpha, void *cuda_stream,
                      int32_t *out_class, double *out_radius, int32_t *out_counts0, int32_t *out_counts)
{
    if (!m || !x_u8 || !out_class || !out_radius || n_images < 0) return ISC_ERR_ARG;
    if (N0 < 1 || N < 1 || !(alpha > 0.0 && alpha < 1.0)) return ISC_ERR_ARG;
    if (N0 > (1ll << 31) - 1 || N > (1ll << 31) - 1) return ISC_ERR_ARG;
    int rc = check_stream_args(image_id0 + (uint64_t)std::max(n_images - 1, 0), 0, 0, std::max(N0, N), sigma);
    if (rc) return rc;
    if (n_images == 0) return ISC_OK;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t C = (size_t)m->n_classes;
    const size_t d = (size_t)m->in_c * m->in_h * m->in_w;
    if ((rc = ensure_noise_table(m, sigma, st))) return rc;
    if ((rc = ensure_counts(m, 2 * C * (size_t)n_images))) return rc;
    const uint8_t *d_x;
    if ((rc = stage_image(m, x_u8, d * (size_t)n_images, x_on_device != 0, st, &d_x))) return rc;
    CK(cudaMemsetAsync(m->d_counts, 0, 2 * C * (size_t)n_images * sizeof(int32_t), st));
    // Pinned staging for the counts and one event per image: the host bound of image i (Algorithm 1 steps 5-7, up to
    // a hundred milliseconds of bisection at N = 100,000) runs on a worker thread while the kernels of the images
    // after it are in flight.
    const size_t need = 2 * C * (size_t)n_images * sizeof(int32_t);
    if (m->h_counts_bytes < need) {
        if (m->h_counts) cudaFreeHost(m->h_counts);
        m->h_counts = nullptr; m->h_counts_bytes = 0;
        CK(cudaHostAlloc((void **)&m->h_counts, need, cudaHostAllocDefault));
        m->h_counts_bytes = need;
    }
    while ((int)m->events.size() < n_images) {
        cudaEvent_t ev;
        CK(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
        m->events.push_back(ev);
    }
    int dev = 0;
    CK(cudaGetDevice(&dev));
    std::vector<int32_t> cls((size_t)n_images, -1);
    std::vector<double> rad((size_t)n_images, 0.0);
    std::atomic<int> enqueued(0);
    std::atomic<bool> failed(false);
    int32_t *h = m->h_counts;
    const int n_cls = m->n_classes;
    // a few workers, image i on worker i mod n_workers: one bound can take longer than one image's kernels
    const int n_workers = std::max(1, std::min(std::min(n_images, 4), (int)std::thread::hardware_concurrency()));
    auto work = [&, dev, h, n_cls](int first) {
        if (cudaSetDevice(dev) != cudaSuccess) { failed = true; return; }
        for (int i = first; i < n_images; i += n_workers) {
            while (enqueued.load(std::memory_order_acquire) <= i) {
                if (failed.load()) return;
                std::this_thread::yield();
            }
            if (cudaEventSynchronize(m->events[(size_t)i]) != cudaSuccess) { failed = true; return; }
            const int32_t *c0 = h + (size_t)i * 2 * C, *c1 = c0 + C;
            double radius = 0.0;
            cls[(size_t)i] = decide_certify(c0, c1, n_cls, N, sigma, alpha, &radius, nullptr);
            rad[(size_t)i] = radius;
        }
    };
    std::vector<std::thread> workers;
    for (int t = 0; t < n_workers; ++t) workers.emplace_back(work, t);
    for (int i = 0; i < n_images && rc == ISC_OK; ++i) {
        int32_t *c0 = m->d_counts + (size_t)i * 2 * C;
        rc = run_counts(m, d_x + (size_t)i * d, seed, image_id0 + (uint64_t)i, 0, 0, N0, st, c0, nullptr);
        if (rc == ISC_OK)
            rc = run_counts(m, d_x + (size_t)i * d, seed, image_id0 + (uint64_t)i, 1, 0, N, st, c0 + C, nullptr);
        if (rc == ISC_OK && (cudaMemcpyAsync(h + (size_t)i * 2 * C, c0, 2 * C * sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
                             cudaEventRecord(m->events[(size_t)i], st) != cudaSuccess)) {
            cudaGetLastError();
            rc = ISC_ERR_CUDA;
        }
        if (rc == ISC_OK) enqueued.store(i + 1, std::memory_order_release);
    }
    if (rc) failed = true;
    for (std::thread &t : workers) t.join();
    if (rc) { cudaStreamSynchronize(st); return rc; }
    CK(cudaStreamSynchronize(st));
    if (failed.load()) return ISC_ERR_CUDA;
    if ((rc = check_engines(m))) return rc;
    for (int i = 0; i < n_images; ++i) {
        const int32_t *c0 = h + (size_t)i * 2 * C, *c1 = c0 + C;
        out_class[i] = cls[(size_t)i];
        out_radius[i] = rad[(size_t)i];
        if (out_counts0) memcpy(out_counts0 + (size_t)i * C, c0, C * sizeof(int32_t));
        if (out_counts) memcpy(out_counts + (size_t)i * C, c1, C * sizeof(int32_t));
    }
    return ISC_OK;
}

int isc_certify(isc_model *m, const uint8_t *x_u8, uint64_t seed, uint64_t image_id, int64_t N0, int64_t N,
                double sigma, double alpha, void *cuda_stream, int32_t *out_class, double *out_radius,
                int32_t *out_counts0, int32_t *out_counts)
{
    return isc_certify_batch(m, x_u8, 0, 1, seed, image_id, N0, N, sigma, alpha, cuda_stream, out_class,
                             out_radius, out_counts0, out_counts);
}

int isc_decide_certify(const int32_t *counts0, const int32_t *counts, int n_classes, int64_t N, double sigma,
                       double alpha, int32_t *out_class, double *out_radius, double *out_p_lower)
{
    if (!counts0 || !counts || !out_class || !out_radius || n_classes < 1 || N < 1) return ISC_ERR_ARG;
    if (!(alpha > 0.0 && alpha < 1.0) || !(sigma > 0.0)) return ISC_ERR_ARG;
    for (int c = 0; c < n_classes; ++c)
        if (counts0[c] < 0 || counts[c] < 0 || counts[c] > N) return ISC_ERR_ARG;
    double radius = 0.0, pl = 0.0;
    *out_class = decide_certify(counts0, counts, n_classes, N, sigma, alpha, &radius, &pl);
    *out_radius = radius;
    if (out_p_lower) *out_p_lower = pl;
    return ISC_OK;
}

int isc_decide_certify_integer(const int32_t *counts0, const int32_t *counts, int n_classes, int64_t N, double sigma,
                               double alpha, int two_sided, int32_t *out_class, int32_t *out_q, int64_t *out_q_squared)
{
    if (!counts0 || !counts || !out_class || !out_q || n_classes < 1 || N < 1) return ISC_ERR_ARG;
    if (!(alpha > 0.0 && alpha < 1.0) || !(sigma > 0.0) || !std::isfinite(sigma) || sigma > 64.0) return ISC_ERR_ARG;
    for (int c = 0; c < n_classes; ++c)
        if (counts0[c] < 0 || counts[c] < 0 || counts[c] > N) return ISC_ERR_ARG;
    int32_t q = 0;
    int64_t q2 = 0;
    *out_class = decide_certify_integer(counts0, counts, n_classes, N, sigma, alpha, two_sided != 0, &q, &q2);
    *out_q = q;
    if (out_q_squared) *out_q_squared = q2;
    return ISC_OK;
}

int isc_certify_integer(isc_model *m, const uint8_t *x_u8, uint64_t seed, uint64_t image_id, int64_t N0, int64_t N,
                        double sigma, double alpha, int two_sided, void *cuda_stream, int32_t *out_class,
                        int32_t *out_q, int64_t *out_q_squared, int32_t *out_counts0, int32_t *out_counts)
{
    if (!m || !x_u8 || !out_class || !out_q) return ISC_ERR_ARG;
    const size_t C = (size_t)m->n_classes;
    std::vector<int32_t> c0(C), c1(C);
    int32_t cls = -1;
    double radius = 0.0;
    int rc = isc_certify_batch(m, x_u8, 0, 1, seed, image_id, N0, N, sigma, alpha, cuda_stream, &cls, &radius,
                               c0.data(), c1.data());
    if (rc) return rc;
    rc = isc_decide_certify_integer(c0.data(), c1.data(), m->n_classes, N, sigma, alpha, two_sided, &cls, out_q, out_q_squared);
    if (rc) return rc;
    *out_class = cls;
    if (out_counts0) memcpy(out_counts0, c0.data(), C * sizeof(int32_t));
    if (out_counts) memcpy(out_counts, c1.data(), C * sizeof(int32_t));
    return ISC_OK;
}

int isc_decide_predict(const int32_t *counts, int n_classes, double alpha, int32_t *out_class)
{
    if (!counts || !out_class || n_classes < 1 || !(alpha > 0.0 && alpha < 1.0)) return ISC_ERR_ARG;
    for (int c = 0; c < n_classes; ++c)
        if (counts[c] < 0) return ISC_ERR_ARG;
    *out_class = decide_predict(counts, n_classes, alpha);
    return ISC_OK;
}

int isc_noise_table(double sigma, uint32_t *cum, int64_t capacity, int32_t *out_T)
{
    if (!out_T || !(sigma > 0.0) || !std::isfinite(sigma) || sigma > 64.0) return ISC_ERR_ARG;
    const int T = noise_halfwidth(sigma);
    if (cum) {
        if (capacity < 2 * (int64_t)T + 1) return ISC_ERR_ARG;
        std::vector<uint32_t> t;
        noise_table(sigma, t);
        memcpy(cum, t.data(), t.size() * sizeof(uint32_t));
    }
    *out_T = T;
    return ISC_OK;
}

int isc_noise_table_rounded(double sigma, uint32_t *cum, int64_t capacity, int32_t *out_T)
{
    if (!out_T || !(sigma > 0.0) || !std::isfinite(sigma) || sigma > 64.0) return ISC_ERR_ARG;
    const int T = noise_halfwidth(sigma);
    if (cum) {
        if (capacity < 2 * (int64_t)T + 1) return ISC_ERR_ARG;
        std::vector<uint32_t> t;
        noise_table_rounded(sigma, t);
        memcpy(cum, t.data(), t.size() * sizeof(uint32_t));
    }
    *out_T = T;
    return ISC_OK;
}

int isc_certified_metrics(const int32_t *classes, const double *radii, const int32_t *labels, int64_t n,
                          const double *r, int n_r, double *out_cp, double *out_ca)
{
    if (!out_cp || n < 0 || n_r < 0 || (n > 0 && (!classes || !radii || !labels)) || (n_r > 0 && (!r || !out_ca)))
        return ISC_ERR_ARG;
    int64_t certified = 0;
    for (int64_t i = 0; i < n; ++i) certified += classes[i] != -1;
    std::vector<double> ca((size_t)n_r, 0.0);
    for (int t = 0; t < n_r; ++t) {
        int64_t hit = 0;
        for (int64_t i = 0; i < n; ++i) hit += classes[i] != -1 && classes[i] == labels[i] && radii[i] >= r[t];
        ca[(size_t)t] = certified ? (double)hit / (double)certified : 0.0;
    }
    *out_cp = n ? (double)certified / (double)n : 0.0;
    for (int t = 0; t < n_r; ++t) out_ca[t] = ca[(size_t)t];
    return ISC_OK;
}

int isc_radius_integer(double sigma, uint32_t p_fx, int32_t *out_q, int64_t *out_q_squared)
{
    if (!out_q || !(sigma > 0.0) || !std::isfinite(sigma) || sigma > 64.0) return ISC_ERR_ARG;
    std::vector<uint32_t> t;
    noise_table(sigma, t);
    const int32_t T = (int32_t)(t.size() - 1) / 2;
    // the table is non-decreasing: first entry that reaches p_fx
    const int32_t q = (int32_t)(std::lower_bound(t.begin(), t.end(), p_fx) - t.begin());
    const int32_t level = q > 2 * T ? T : q - T;
    *out_q = level;
    if (out_q_squared) *out_q_squared = (int64_t)level * (int64_t)level;
    return ISC_OK;
}

int isc_debug_tensor(isc_model *m, const uint8_t *x_u8, uint64_t seed, uint64_t image_id, int32_t phase,
                     int64_t j, double sigma, int tensor, void *cuda_stream, int32_t *out, int64_t capacity)
{
    if (!m || !x_u8 || !out || tensor < 0 || tensor > (int)m->layers.size()) return ISC_ERR_ARG;
    int rc = check_stream_args(image_id, phase, j, 1, sigma);
    if (rc) return rc;
    const TShape &s = m->shapes[(size_t)tensor];
    const size_t n = (size_t)s.c * s.h * s.w;
    if (capacity < (int64_t)n) return ISC_ERR_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if ((rc = ensure_noise_table(m, sigma, st))) return rc;
    const uint8_t *d_x;
    if ((rc = stage_image(m, x_u8, (size_t)m->in_c * m->in_h * m->in_w, false, st, &d_x))) return rc;
    NoiseStream ns = make_stream(m, seed, image_id, phase, j);
    if (m->opt_engine == 3) {       // read the tensor back from the resident engine
        if (!m->line) return ISC_ERR_UNSUPPORTED;
        if ((rc = ensure_counts(m, (size_t)m->n_classes))) return rc;
        std::vector<int32_t> tmp(n);
        rc = isc::line_debug_tensor(m->line, d_x, ns, tensor, tmp.data(), m->d_counts, st, &m->launches);
        if (rc) return rc;
        memcpy(out, tmp.data(), n * sizeof(int32_t));
        return ISC_OK;
    }
    if (tensor == 0) {
        int32_t *d_out = nullptr;
        CK(cudaMalloc((void **)&d_out, n * sizeof(int32_t)));
        cudaError_t e = launch_noisy_input(d_x, m->in_c, m->in_h, m->in_w, ns, 1, d_out, st);
        m->launches += 1;
        if (e == cudaSuccess) e = cudaMemcpyAsync(out, d_out, n * sizeof(int32_t), cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        cudaFree(d_out);
        return e == cudaSuccess ? ISC_OK : ISC_ERR_CUDA;
    }
    if ((rc = ensure_workspace(m, 1))) return rc;
    if ((rc = generic_forward(m, d_x, ns, 1, st, tensor - 1, m->opt_engine == 2 || (m->opt_engine == 0 && m->has_tc)))) return rc;
    std::vector<int8_t> h((size_t)s.h * s.w * s.cp);
    CK(cudaMemcpyAsync(h.data(), m->bufs[(size_t)m->tensor_buf[(size_t)tensor]].p, h.size(),
                       cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    for (int c = 0; c < s.c; ++c)
        for (int y = 0; y < s.h; ++y)
            for (int x = 0; x < s.w; ++x)
                out[((size_t)c * s.h + y) * s.w + x] = h[((size_t)y * s.w + x) * s.cp + c];
    return ISC_OK;
}

int isc_debug_residual_form(int32_t res_mult, int32_t res_shift, int32_t zp_res, int32_t *k, int32_t *c)
{
    if (!k || !c) return ISC_ERR_ARG;
    uint32_t k8 = 0;
    int32_t cc = 0;
    if (!isc::residual_short_form(res_mult, res_shift, zp_res, &k8, &cc)) return 0;
    *k = (int32_t)(k8 >> 8);
    *c = cc;
    return 1;
}

int isc_debug_wait_timeout(isc_model *m, int64_t limit_ns, void *cuda_stream, int32_t *out4)
{
    if (!m || !out4) return ISC_ERR_ARG;
    if (!m->line && m->has_tc) {
        // The layer-by-layer tensor-core engine: one launch of its first implicit-GEMM layer on one sample's work
        // space with the weights held back, so that the kernel's own waits run out and its CTAs leave through the
        // abort path; the error word must be up afterwards.
        cudaStream_t st = (cudaStream_t)cuda_stream;
        size_t li = 1;
        while (li < m->glayers.size() && !m->wpacks[li]) ++li;
        if (li >= m->glayers.size()) return ISC_ERR_UNSUPPORTED;
        int rc = ensure_workspace(m, 1);
        if (rc) return rc;
        const GLayer &G = m->glayers[li];
        const isc_layer &L = m->layers[li].d;
        int8_t *out = (int8_t *)m->bufs[(size_t)m->tensor_buf[li + 1]].p;
        const int8_t *in = (const int8_t *)m->bufs[(size_t)m->tensor_buf[(size_t)L.in_tensor]].p;
        const int8_t *res = L.res_tensor >= 0 ? (const int8_t *)m->bufs[(size_t)m->tensor_buf[(size_t)L.res_tensor]].p : nullptr;
        const auto t0 = std::chrono::steady_clock::now();
        if (launch_igemm_conv(G, m->wpacks[li], m->tc_cst[li], m->tc_fast[li] != 0, m->tc_resk[li], 1, in, res, out, m->d_tc_err, st, true) != cudaSuccess)
            return ISC_ERR_CUDA;
        CK(cudaStreamSynchronize(st));
        const long long ns = std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - t0).count();
        int32_t e = 0;
        CK(cudaMemcpy(&e, m->d_tc_err, sizeof(e), cudaMemcpyDeviceToHost));
        CK(cudaMemset(m->d_tc_err, 0, sizeof(e)));
        out4[0] = 0; out4[1] = 0; out4[2] = e; out4[3] = (int32_t)std::min<long long>(ns, 0x7FFFFFFF);
        return e != 0 ? ISC_ERR_TIMEOUT : ISC_OK;
    }
    if (!m->line) return ISC_ERR_UNSUPPORTED;
    int32_t tmp[4] = {0, 0, 0, 0};
    const int rc = isc::line_wait_probe(m->line, limit_ns, tmp, (cudaStream_t)cuda_stream);
    if (rc == ISC_ERR_ARG || rc == ISC_ERR_CUDA) return rc;
    memcpy(out4, tmp, sizeof(tmp));
    return rc;
}

}  // extern "C"

// ------------------------------------------------------------------ allocation-free variant
//
// Work space of isc_sample_counts_static: one fixed array in the library's device image.  Every
// GPU on which the library is loaded carries it from module load until the process exits.
#define ISC_STATIC_SCRATCH_BYTES (32u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[ISC_STATIC_SCRATCH_BYTES];

namespace {

constexpr size_t kStaticCountsBytes = 16u << 10;     // up to 4096 classes
constexpr size_t kStaticTableBytes = 64u << 10;      // up to 16384 table entries (sigma up to ~4.5)
constexpr size_t kStaticImageBytes = 1u << 20;       // up to 1 MiB of input image
constexpr int kMaxDevices = 64;
unsigned char *g_static_ptr[kMaxDevices];            // device address of the array, per device ordinal

// The symbol name is only a host-side handle; the kernels need the array's device address,
// which the runtime reports per device.  Done once for each device, with that device current.
int static_scratch_base(unsigned char **base)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ISC_ERR_CUDA;
    if (!g_static_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return ISC_ERR_CUDA;
        }
        g_static_ptr[dev] = static_cast<unsigned char *>(p);
    }
    *base = g_static_ptr[dev];
    return ISC_OK;
}

}  // namespace

extern "C" int isc_sample_counts_static(isc_model *m, const uint8_t *x_u8, uint64_t seed, uint64_t image_id,
                                        int32_t phase, int64_t first_sample, int64_t n_samples, double sigma,
                                        void *cuda_stream, int32_t *out_counts)
{
    if (!m || !x_u8 || !out_counts) return ISC_ERR_ARG;
    int rc = check_stream_args(image_id, phase, first_sample, n_samples, sigma);
    if (rc) return rc;
    if (n_samples > (1ll << 31) - 1) return ISC_ERR_ARG;
    const size_t C = (size_t)m->n_classes;
    const size_t d = (size_t)m->in_c * m->in_h * m->in_w;
    const int T = noise_halfwidth(sigma);
    const size_t per_sample = generic_bytes_per_sample(m) + 256 * m->buf_bytes.size();
    const size_t fixed = kStaticCountsBytes + kStaticTableBytes + kStaticImageBytes;
    // sizes beyond the fixed work space are refused, never silently truncated
    if (C * sizeof(int32_t) > kStaticCountsBytes) return ISC_ERR_UNSUPPORTED;
    if ((size_t)(2 * T + 1) * sizeof(uint32_t) > kStaticTableBytes) return ISC_ERR_UNSUPPORTED;
    if (d > kStaticImageBytes) return ISC_ERR_UNSUPPORTED;
    if (per_sample > ISC_STATIC_SCRATCH_BYTES - fixed) return ISC_ERR_UNSUPPORTED;

    unsigned char *base = nullptr;
    if ((rc = static_scratch_base(&base))) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int32_t *d_counts = reinterpret_cast<int32_t *>(base);
    uint32_t *d_cum = reinterpret_cast<uint32_t *>(base + kStaticCountsBytes);
    uint8_t *d_x = base + kStaticCountsBytes + kStaticTableBytes;
    unsigned char *act = base + fixed;
    const int64_t cap = std::min<int64_t>(32768, (int64_t)((ISC_STATIC_SCRATCH_BYTES - fixed) / per_sample));

    // carve the activation buffers for `cap` samples out of the array (256-byte aligned)
    std::vector<int8_t *> buf(m->buf_bytes.size());
    size_t off = 0;
    for (size_t b = 0; b < buf.size(); ++b) {
        buf[b] = reinterpret_cast<int8_t *>(act + off);
        off += (m->buf_bytes[b] * (size_t)cap + 255) & ~(size_t)255;
    }

    std::vector<uint32_t> cum;
    if (m->opt_noise) noise_table_rounded(sigma, cum); else noise_table(sigma, cum);
    m->last_engine = 1;
    // the array keeps whatever the previous call left: the vote counts must start from zero
    CK(cudaMemsetAsync(d_counts, 0, C * sizeof(int32_t), st));
    CK(cudaMemcpyAsync(d_cum, cum.data(), cum.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, st));
    CK(cudaMemcpyAsync(d_x, x_u8, d, cudaMemcpyHostToDevice, st));
    const int n_layers = (int)m->glayers.size();
    for (int64_t done = 0; done < n_samples; done += cap) {
        const int b = (int)std::min<int64_t>(cap, n_samples - done);
        NoiseStream ns = make_stream(m, seed, image_id, phase, first_sample + done);
        ns.cum = d_cum;
        ns.T = T;
        ns.guide = nullptr;
        ns.guide_steps = 0;
        for (int i = 0; i < n_layers; ++i) {
            const GLayer &G = m->glayers[(size_t)i];
            const isc_layer &L = m->layers[(size_t)i].d;
            int8_t *out = buf[(size_t)m->tensor_buf[(size_t)i + 1]];
            const int8_t *in = i == 0 ? nullptr : buf[(size_t)m->tensor_buf[(size_t)L.in_tensor]];
            const int8_t *res = L.res_tensor >= 0 ? buf[(size_t)m->tensor_buf[(size_t)L.res_tensor]] : nullptr;
            cudaError_t e;
            if (i == 0) e = launch_first_conv(G, d_x, m->in_c, ns, b, out, st);
            else if (L.op == ISC_CONV2D || L.op == ISC_FC) e = launch_conv(G, b, in, res, out, st);
            else if (L.op == ISC_GAVGPOOL) e = launch_gavgpool(G, b, in, out, st);
            else e = launch_maxpool(G, b, in, out, st);
            m->launches += 1;
            if (e != cudaSuccess) { cudaStreamSynchronize(st); return ISC_ERR_CUDA; }
        }
        cudaError_t e = launch_votes(buf[(size_t)m->tensor_buf[(size_t)n_layers]], m->shapes[(size_t)n_layers].cp,
                                     m->n_classes, b, d_counts, nullptr, st);
        m->launches += 1;
        if (e != cudaSuccess) { cudaStreamSynchronize(st); return ISC_ERR_CUDA; }
    }
    std::vector<int32_t> h(C);
    CK(cudaMemcpyAsync(h.data(), d_counts, C * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    memcpy(out_counts, h.data(), C * sizeof(int32_t));
    return ISC_OK;
}

extern "C" {

int isc_set_option(isc_model *m, const char *name, int64_t value)
{
    if (!m || !name) return ISC_ERR_ARG;
    if (!strcmp(name, "batch")) {
        if (value < 0 || value > (1 << 20)) return ISC_ERR_ARG;
        m->opt_batch = value;
        return ISC_OK;
    }
    if (!strcmp(name, "noise")) {
        if (value != 0 && value != 1) return ISC_ERR_ARG;
        m->opt_noise = value;
        return ISC_OK;
    }
    if (!strcmp(name, "tensor_copy")) {
        if (value != 0 && value != 1) return ISC_ERR_ARG;
        m->opt_tensor_copy = value;
        return ISC_OK;
    }
    if (!strcmp(name, "engine")) {
        if (value < 0 || value > 3) return ISC_ERR_ARG;
        m->opt_engine = value;
        return ISC_OK;
    }
    return ISC_ERR_ARG;
}

int isc_get_info(isc_model *m, const char *name, int64_t *out)
{
    if (!m || !name || !out) return ISC_ERR_ARG;
    if (!strcmp(name, "engine")) *out = m->last_engine;
    else if (!strcmp(name, "gpu_launches")) *out = m->launches;
    else if (!strcmp(name, "macs_per_sample")) *out = m->macs;
    else if (!strcmp(name, "has_line_engine")) *out = m->line ? 1 : 0;
    else if (!strcmp(name, "has_tensor_core_layers")) *out = m->has_tc ? 1 : 0;
    else if (!strncmp(name, "cycles_", 7)) {
        static const char *const which[4] = {"cycles_fill", "cycles_noise", "cycles_conv", "cycles_tail"};
        if (!m->line) return ISC_ERR_UNSUPPORTED;
        unsigned long long c[4];
        int rc = isc::line_phase_cycles(m->line, c);
        if (rc) return rc;
        for (int k = 0; k < 4; ++k)
            if (!strcmp(name, which[k])) { *out = (int64_t)c[k]; return ISC_OK; }
        return ISC_ERR_ARG;
    }
    else return ISC_ERR_ARG;
    return ISC_OK;
}

}  // extern "C"
