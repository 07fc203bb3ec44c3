/*
 * fp64 CPU oracle for mixed-tenant batched inference.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code, header, table or
 * helper with the CUDA path and must never be called from it.
 *
 * What it computes, and where the paper says so:
 *   - A DNN is a stateless, deterministic function of (weights, input)
 *     (Sec. 1.1): orc_forward_one depends on nothing but its arguments.
 *   - A DNN is evaluated one layer after the other, each layer's operation
 *     applied to the previous layer's output (Sec. 1.1): the loop over layers
 *     below, no fusion, no reordering.
 *   - A fully-connected layer multiplies the previous layer's output by a
 *     tensor of learned constants (Sec. 1.1).  Reading used here (the paper
 *     gives no orientation or bias): z = W a + b, W stored [out][in].
 *   - A worker hosts the DNNs of many tenants and receives requests, each for
 *     one model (Sec. 3): orc_forward_batch evaluates request i with the
 *     layers of models[ids[i]], one request at a time, independent of every
 *     other request in the batch.
 *   - Grouping requests by model is a pure re-ordering; its unique stable
 *     form is a counting sort: orc_bucket.
 *
 * The conv, pooling and ReLU layers are not defined by the paper (it only
 * names a catalogue of standard layer types, Sec. 1.1 / Sec. 3.1); they follow
 * the textbook definitions:
 *   conv3x3: cross-correlation, stride 1, zero padding 1, NHWC activations,
 *            weights [out][ky][kx][in]; tap (ky,kx) reads pixel (y+ky-1, x+kx-1)
 *   conv1x1: the fully-connected layer applied at every pixel, NHWC,
 *            weights [out][in]: z[p][o] = b[o] + sum_c W[o][c] a[p][c]
 *   global average pool: mean over all H*W positions, per channel
 *   ReLU: max(z, 0)
 *   identity shortcut (the residual block of the network the paper uses as
 *            its running example, Sec. 1.1: resnet18): a conv layer marked
 *            `residual` adds the INPUT of the layer before it to its own
 *            pre-activation, a_{l+1} = act(conv(a_l) + b + a_{l-1}), which
 *            closes a block of two conv layers
 *
 * Precision: every value is held in double from the bf16 input to the output;
 * nothing is rounded between layers.  bf16 and fp32 inputs are exact in double.
 *
 * Parity pins (tests that do not go through this file's own formulas):
 * identity and zero weights (closed forms), a separately written triple-loop
 * matmul, numpy float64 matmul, brute-force padded-copy conv, scipy
 * correlate2d, shifted-tap and all-ones closed forms, numpy stable argsort and
 * an O(n*T) brute-force bucketing; conv1x1 by the dense layer applied pixel
 * by pixel and by a conv3x3 whose only non-zero tap is the centre one; the
 * shortcut by a zero-weight block
 * (a closed form of the block's input alone) and a scipy restatement.
 * No function here is left unpinned.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_DENSE = 0, ORC_CONV3X3 = 1, ORC_GLOBAL_AVG_POOL = 2, ORC_CONV1X1 = 3 };

typedef struct {
    int32_t kind;
    int32_t in_ch, out_ch;
    int32_t h, w;          /* spatial size for conv / pool; 0 for dense */
    int32_t relu;          /* 1: apply max(z,0) after the layer */
    int32_t residual;      /* conv only, 1: add the previous layer's input before the activation */
    const uint16_t* weight; /* bf16 bit patterns; NULL for pool */
    const float* bias;      /* fp32 [out_ch]; NULL means zeros */
} orc_layer;

static double bf16_to_double(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static int64_t layer_in_elems(const orc_layer* l)
{
    return l->kind == ORC_DENSE ? (int64_t)l->in_ch : (int64_t)l->in_ch * l->h * l->w;
}

static int64_t layer_out_elems(const orc_layer* l)
{
    return (l->kind == ORC_CONV3X3 || l->kind == ORC_CONV1X1) ? (int64_t)l->out_ch * l->h * l->w : (int64_t)l->out_ch;
}

/* Stable counting sort of request indices by model id.
 *   counts[t]   = number of requests with id t
 *   offsets[0]  = 0, offsets[t+1] = offsets[t] + counts[t]      (size T+1)
 *   perm[j]     = arrival index of the request at bucketed position j
 *                 (ascending arrival index inside each segment)
 *   inv[i]      = bucketed position of arrival index i
 * Returns 0, or -1 if an id is outside [0, T). */
int orc_bucket(const int32_t* ids, int32_t n, int32_t T,
               int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv)
{
    for (int32_t t = 0; t < T; ++t) counts[t] = 0;
    for (int32_t i = 0; i < n; ++i) {
        if (ids[i] < 0 || ids[i] >= T) return -1;
        counts[ids[i]] += 1;
    }
    offsets[0] = 0;
    for (int32_t t = 0; t < T; ++t) offsets[t + 1] = offsets[t] + counts[t];
    int32_t* next = (int32_t*)malloc(sizeof(int32_t) * (size_t)(T > 0 ? T : 1));
    if (!next) return -2;
    for (int32_t t = 0; t < T; ++t) next[t] = offsets[t];
    for (int32_t i = 0; i < n; ++i) {
        int32_t pos = next[ids[i]]++;
        perm[pos] = i;
        inv[i] = pos;
    }
    free(next);
    return 0;
}

/* One layer: a (in) -> z (out), both double.  skip: the tensor a residual
 * layer adds before its activation (same shape as z), else NULL. */
static void layer_apply(const orc_layer* l, const double* a, const double* skip, double* z)
{
    if (l->kind == ORC_DENSE) {
        for (int32_t o = 0; o < l->out_ch; ++o) {
            double acc = l->bias ? (double)l->bias[o] : 0.0;
            const uint16_t* wrow = l->weight + (int64_t)o * l->in_ch;
            for (int32_t k = 0; k < l->in_ch; ++k)
                acc += bf16_to_double(wrow[k]) * a[k];
            z[o] = acc;
        }
    } else if (l->kind == ORC_CONV3X3) {
        const int32_t H = l->h, W = l->w, C = l->in_ch, O = l->out_ch;
        for (int32_t y = 0; y < H; ++y)
            for (int32_t x = 0; x < W; ++x)
                for (int32_t o = 0; o < O; ++o) {
                    double acc = l->bias ? (double)l->bias[o] : 0.0;
                    for (int32_t ky = 0; ky < 3; ++ky) {
                        const int32_t yy = y + ky - 1;
                        if (yy < 0 || yy >= H) continue;      /* zero padding */
                        for (int32_t kx = 0; kx < 3; ++kx) {
                            const int32_t xx = x + kx - 1;
                            if (xx < 0 || xx >= W) continue;  /* zero padding */
                            const uint16_t* wv = l->weight + (((int64_t)o * 3 + ky) * 3 + kx) * C;
                            const double* av = a + ((int64_t)yy * W + xx) * C;
                            for (int32_t c = 0; c < C; ++c)
                                acc += bf16_to_double(wv[c]) * av[c];
                        }
                    }
                    z[((int64_t)y * W + x) * O + o] = acc;
                }
    } else if (l->kind == ORC_CONV1X1) {
        const int64_t P = (int64_t)l->h * l->w;
        for (int64_t p = 0; p < P; ++p)
            for (int32_t o = 0; o < l->out_ch; ++o) {
                double acc = l->bias ? (double)l->bias[o] : 0.0;
                const uint16_t* wrow = l->weight + (int64_t)o * l->in_ch;
                const double* av = a + p * l->in_ch;
                for (int32_t c = 0; c < l->in_ch; ++c)
                    acc += bf16_to_double(wrow[c]) * av[c];
                z[p * l->out_ch + o] = acc;
            }
    } else { /* global average pool */
        const int64_t P = (int64_t)l->h * l->w;
        for (int32_t c = 0; c < l->in_ch; ++c) {
            double s = 0.0;
            for (int64_t p = 0; p < P; ++p) s += a[p * l->in_ch + c];
            z[c] = s / (double)P;
        }
    }
    if (skip) {
        const int64_t n_out = layer_out_elems(l);
        for (int64_t j = 0; j < n_out; ++j) z[j] += skip[j];
    }
    if (l->relu) {
        const int64_t n_out = layer_out_elems(l);
        for (int64_t j = 0; j < n_out; ++j)
            if (z[j] < 0.0) z[j] = 0.0;
    }
}

/* Forward pass of one request through one model.  out must hold the last
 * layer's out_elems doubles.  Returns 0, -1 on a shape-chain mismatch, -2 on
 * allocation failure. */
int orc_forward_one(const orc_layer* layers, int32_t n_layers, const uint16_t* input, double* out)
{
    if (n_layers <= 0) return -1;
    int64_t max_elems = layer_in_elems(&layers[0]);
    for (int32_t li = 0; li < n_layers; ++li) {
        if (li > 0 && layer_in_elems(&layers[li]) != layer_out_elems(&layers[li - 1])) return -1;
        if (layer_out_elems(&layers[li]) > max_elems) max_elems = layer_out_elems(&layers[li]);
        if (layers[li].residual) {
            /* the shortcut joins the output of this layer with the input of the one before: both are conv
             * layers and the three tensors have one shape */
            if (li == 0 || layers[li].kind != ORC_CONV3X3 || layers[li - 1].kind != ORC_CONV3X3) return -1;
            if (layer_in_elems(&layers[li - 1]) != layer_out_elems(&layers[li])) return -1;
        }
    }
    /* three tensors are alive at a time: the previous layer's input, this layer's input, its output */
    double* before = (double*)malloc(sizeof(double) * (size_t)max_elems);
    double* a = (double*)malloc(sizeof(double) * (size_t)max_elems);
    double* z = (double*)malloc(sizeof(double) * (size_t)max_elems);
    if (!before || !a || !z) { free(before); free(a); free(z); return -2; }
    const int64_t n_in = layer_in_elems(&layers[0]);
    for (int64_t j = 0; j < n_in; ++j) a[j] = bf16_to_double(input[j]);
    for (int32_t li = 0; li < n_layers; ++li) {
        layer_apply(&layers[li], a, layers[li].residual ? before : NULL, z);
        double* t = before; before = a; a = z; z = t;
    }
    const int64_t n_out = layer_out_elems(&layers[n_layers - 1]);
    for (int64_t j = 0; j < n_out; ++j) out[j] = a[j];
    free(before); free(a); free(z);
    return 0;
}

/* The mixed batch: request i is evaluated by models[ids[i]] on inputs[i, :].
 * Requests are independent; the loop over them may run on several threads.
 * Returns 0 or the first non-zero code met (-1 shape/id, -2 alloc). */
int orc_forward_batch(const orc_layer* const* models, const int32_t* n_layers, int32_t T,
                      const int32_t* ids, int32_t n,
                      const uint16_t* inputs, int64_t in_elems,
                      double* out, int64_t out_elems, int32_t n_threads)
{
    int rc = 0;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#else
    (void)n_threads;
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t i = 0; i < n; ++i) {
        int r;
        const int32_t t = ids[i];
        if (t < 0 || t >= T) {
            r = -1;
        } else if (layer_in_elems(&models[t][0]) != in_elems ||
                   layer_out_elems(&models[t][n_layers[t] - 1]) != out_elems) {
            r = -1;
        } else {
            r = orc_forward_one(models[t], n_layers[t], inputs + (int64_t)i * in_elems,
                                out + (int64_t)i * out_elems);
        }
        if (r != 0) {
#pragma omp critical
            { if (rc == 0) rc = r; }
        }
    }
    return rc;
}

int orc_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
