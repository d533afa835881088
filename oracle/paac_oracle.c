/*
 * PAAC oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow CPU statement of one parallel advantage actor-critic
 * iteration (Algorithm 1 of the paper, with the gradients of Section 4,
 * Eqs. 9-10) over a seeded synthetic hashed environment.  It exists only to
 * check the CUDA library and to be timed beside it; the library never calls
 * it and the two share no code.
 *
 * Arithmetic convention: every dot product and reduction accumulates in
 * double in a fixed index order; each tensor is rounded to float when it is
 * stored.  With bf16 != 0 the weights used in contractions and the stored
 * activations / activation gradients are additionally rounded to bfloat16
 * (round to nearest even); biases, logits, values, losses, returns and the
 * optimiser stay float.
 *
 * What pins each function (tests/test_oracle_*.py):
 *   philox4x32_10        published known-answer vectors + second implementation
 *   environment hash     second independent implementation + frequencies
 *   forward / backward   PyTorch float64 conv2d/linear + autograd, finite
 *                        differences of the scalar loss, hand cases
 *   softmax / sampling   sum-to-one, entropy bounds, shift invariance, brute force
 *   returns              closed form sum gamma^k r + gamma^n V, worked cases
 *   clip / RMSProp       closed forms
 *   pre-processing       block means of an integer-upsampled image (independent definition),
 *                        pure-colour and constant images, hand-computed rows, channel shift
 *   frame stack          equals the pre-processing's own stacking, known planes in order, restart, brute force
 *   n-step Q variant     brute-force arg max and exploration branch, exploration frequency,
 *                        PyTorch autograd and central differences of the loss, hand case
 * The whole iteration has no printed value in the paper to compare with:
 * beyond the pieces above it is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ */
/* Network description (layer sizes are data, so tiny nets can be tested) */
/* ------------------------------------------------------------------ */
#define ORC_MAX_CONV 4
typedef struct {
  int in_h, in_w, in_c;            /* input frame, NHWC, uint8 */
  int n_conv;                      /* number of conv layers (VALID padding) */
  int cout[ORC_MAX_CONV];
  int k[ORC_MAX_CONV];             /* square kernel */
  int stride[ORC_MAX_CONV];
  int fc;                          /* hidden units of the fully connected layer */
  int n_actions;                   /* policy head width; value head width is 1 */
} orc_net;

static int conv_out(int in, int k, int s) { return (in - k) / s + 1; }

/* shape of conv layer l's input (l = n_conv gives the fc input) */
static void layer_in_shape(const orc_net* n, int l, int* h, int* w, int* c) {
  int H = n->in_h, W = n->in_w, C = n->in_c;
  for (int i = 0; i < l; ++i) {
    H = conv_out(H, n->k[i], n->stride[i]);
    W = conv_out(W, n->k[i], n->stride[i]);
    C = n->cout[i];
  }
  *h = H; *w = W; *c = C;
}

/* Canonical parameter layout: conv1..convL, fc, policy head, value head;
 * each layer W then b; conv W[cout][kh][kw][cin]; fc W[out][in], in = (h,w,c). */
static size_t off_conv_w(const orc_net* n, int l) {
  size_t o = 0;
  for (int i = 0; i < l; ++i) {
    int h, w, c; layer_in_shape(n, i, &h, &w, &c);
    o += (size_t)n->cout[i] * n->k[i] * n->k[i] * c + n->cout[i];
  }
  return o;
}
static size_t conv_w_size(const orc_net* n, int l) {
  int h, w, c; layer_in_shape(n, l, &h, &w, &c);
  return (size_t)n->cout[l] * n->k[l] * n->k[l] * c;
}
static size_t fc_in(const orc_net* n) {
  int h, w, c; layer_in_shape(n, n->n_conv, &h, &w, &c);
  return (size_t)h * w * c;
}
static size_t off_fc_w(const orc_net* n) { return off_conv_w(n, n->n_conv); }
static size_t off_pi_w(const orc_net* n) { return off_fc_w(n) + fc_in(n) * n->fc + n->fc; }
static size_t off_v_w(const orc_net* n) { return off_pi_w(n) + (size_t)n->n_actions * n->fc + n->n_actions; }

size_t orc_param_count(const orc_net* n) { return off_v_w(n) + n->fc + 1; }

/* element count of activation l per state: l < n_conv conv outputs, l == n_conv fc output */
size_t orc_act_size(const orc_net* n, int l) {
  if (l == n->n_conv) return (size_t)n->fc;
  int h, w, c; layer_in_shape(n, l + 1, &h, &w, &c);
  return (size_t)h * w * c;
}

/* ------------------------------------------------------------------ */
/* bfloat16 rounding (round to nearest, ties to even)                   */
/* ------------------------------------------------------------------ */
float orc_bf16_round(float x) {
  uint32_t u; memcpy(&u, &x, 4);
  if ((u & 0x7F800000u) == 0x7F800000u) return x;      /* inf / nan unchanged */
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  u &= 0xFFFF0000u;
  float y; memcpy(&y, &u, 4);
  return y;
}
static float rnd(float x, int bf16) { return bf16 ? orc_bf16_round(x) : x; }

/* ------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: */
/* as easy as 1, 2, 3", SC'11) -- the counter-based generator both the  */
/* initialiser and the action sampler draw from.                        */
/* ------------------------------------------------------------------ */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int r = 0; r < 10; ++r) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

#define STREAM_INIT   1u
#define STREAM_ACTION 2u

static float philox_uniform(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t stream, uint64_t seed) {
  uint32_t ctr[4] = {c0, c1, c2, stream};
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t out[4];
  orc_philox4x32_10(ctr, key, out);
  return (float)(out[0] >> 8) * (1.0f / 16777216.0f);   /* 24 bits -> [0,1) exactly */
}

/* uniform that decides the action of environment env at its global step index */
float orc_action_uniform(uint64_t seed, uint32_t env, uint64_t step) {
  return philox_uniform(env, (uint32_t)step, (uint32_t)(step >> 32), STREAM_ACTION, seed);
}

/* ------------------------------------------------------------------ */
/* Initialisation (Algorithm 1, first line): Xavier-uniform weights,    */
/* zero biases.                                                         */
/* ------------------------------------------------------------------ */
static void xavier_fill(float* w, size_t count, double fan_in, double fan_out, uint32_t layer_id, uint64_t seed) {
  float bound = (float)sqrt(6.0 / (fan_in + fan_out));
  for (size_t i = 0; i < count; ++i) {
    float u = philox_uniform((uint32_t)i, layer_id, 0u, STREAM_INIT, seed);
    w[i] = (2.0f * u - 1.0f) * bound;     /* 2u-1 is exact; one rounding in the product */
  }
}

void orc_init_params(const orc_net* n, uint64_t seed, float* theta) {
  memset(theta, 0, orc_param_count(n) * sizeof(float));
  uint32_t id = 0;
  for (int l = 0; l < n->n_conv; ++l, ++id) {
    int h, w, c; layer_in_shape(n, l, &h, &w, &c);
    double kk = (double)n->k[l] * n->k[l];
    xavier_fill(theta + off_conv_w(n, l), conv_w_size(n, l), kk * c, kk * n->cout[l], id, seed);
  }
  xavier_fill(theta + off_fc_w(n), fc_in(n) * n->fc, (double)fc_in(n), (double)n->fc, id++, seed);
  xavier_fill(theta + off_pi_w(n), (size_t)n->n_actions * n->fc, (double)n->fc, (double)n->n_actions, id++, seed);
  xavier_fill(theta + off_v_w(n), (size_t)n->fc, (double)n->fc, 1.0, id++, seed);
}

/* ------------------------------------------------------------------ */
/* Synthetic hashed environment (stands in for the emulators of         */
/* Algorithm 1's parallel-for: apply a_t, observe s_{t+1}, r, terminal) */
/* Everything is a pure integer function of (seed, env, step, action).  */
/* ------------------------------------------------------------------ */
#define HK0 0x9E3779B9u
#define HK1 0xBB67AE85u
#define HK2 0x6A09E667u
#define TAG_REWARD   0x52455744u
#define TAG_TERMINAL 0x5445524Du

static uint32_t mix(uint32_t x) {
  x ^= x >> 16; x *= HK0; x ^= x >> 15; x *= HK1; x ^= x >> 16;
  return x;
}
static uint32_t env_base(uint64_t seed, uint32_t env, uint32_t step, uint32_t tag) {
  uint32_t h = mix((uint32_t)seed ^ HK2);
  h = mix(h ^ (uint32_t)(seed >> 32));
  h = mix(h ^ env);
  h = mix(h ^ step);
  return mix(h ^ tag);
}

/* frame of the state that environment env is in at step index `step`;
 * tag = 0 for a start state (step 0 or after a terminal), else action+1 of
 * the transition that led here */
void orc_env_frame(uint64_t seed, uint32_t env, uint32_t step, uint32_t tag,
                   int h, int w, uint8_t* frame /* [h][w][4] */) {
  uint32_t base = env_base(seed, env, step, tag);
  for (int y = 0; y < h; ++y)
    for (int x = 0; x < w; ++x) {
      uint32_t word = mix(base + HK0 * (uint32_t)(y * w + x + 1));
      uint8_t* p = frame + ((size_t)y * w + x) * 4;
      p[0] = (uint8_t)word; p[1] = (uint8_t)(word >> 8);
      p[2] = (uint8_t)(word >> 16); p[3] = (uint8_t)(word >> 24);
    }
}

/* reward and terminal flag of taking `action` at step index `step` */
void orc_env_outcome(uint64_t seed, uint32_t env, uint32_t step, int32_t action,
                     uint32_t term_denom, int8_t* reward, uint8_t* terminal) {
  uint32_t base = env_base(seed, env, step, (uint32_t)action + 1u);
  uint32_t hr = mix(base ^ TAG_REWARD) & 15u;
  *reward = hr == 0u ? 1 : (hr == 1u ? -1 : 0);
  uint32_t ht = mix(base ^ TAG_TERMINAL);
  *terminal = (uint8_t)((((uint64_t)ht * term_denom) >> 32) == 0u);
}

void orc_env_reset(uint64_t seed, int n_e, int h, int w, uint8_t* frames) {
  for (int e = 0; e < n_e; ++e)
    orc_env_frame(seed, (uint32_t)e, 0u, 0u, h, w, frames + (size_t)e * h * w * 4);
}

/* one synchronous step of all environments; counters are [n_e] each */
void orc_env_step(uint64_t seed, int n_e, uint32_t step, const int32_t* actions, uint32_t term_denom,
                  int h, int w, uint8_t* next_frames, int8_t* rewards, uint8_t* terminals,
                  int32_t* ep_len, int32_t* ep_return, int32_t* episodes) {
#pragma omp parallel for schedule(static)
  for (int e = 0; e < n_e; ++e) {
    orc_env_outcome(seed, (uint32_t)e, step, actions[e], term_denom, &rewards[e], &terminals[e]);
    uint32_t tag = terminals[e] ? 0u : (uint32_t)actions[e] + 1u;
    orc_env_frame(seed, (uint32_t)e, step + 1u, tag, h, w, next_frames + (size_t)e * h * w * 4);
    ep_len[e] += 1; ep_return[e] += rewards[e];
    if (terminals[e]) { episodes[e] += 1; ep_len[e] = 0; ep_return[e] = 0; }
  }
}

/* ------------------------------------------------------------------ */
/* A second synthetic environment, one a learner can solve (the hashed  */
/* one above has nothing to learn): every state shows which action is   */
/* rewarded.  goal(env, step) = mix(base(env, step, 0) ^ 'GOAL') mod A; */
/* the frame is the hashed frame of the same (env, step, tag) with every */
/* byte reduced to its low six bits (a dim texture, 0..63) and the band */
/* of rows [band * goal, band * (goal + 1)), band = h / A, set to 255   */
/* in all channels; taking action a pays +1 if a is the goal of the     */
/* current state and 0 otherwise; terminals as in the hashed            */
/* environment.  Used for the learning-rate rule of Section 5.3.        */
/* ------------------------------------------------------------------ */
#define TAG_GOAL 0x474F414Cu
uint32_t orc_pattern_goal(uint64_t seed, uint32_t env, uint32_t step, int n_actions) {
  return mix(env_base(seed, env, step, 0u) ^ TAG_GOAL) % (uint32_t)n_actions;
}
void orc_pattern_frame(uint64_t seed, uint32_t env, uint32_t step, uint32_t tag, int n_actions,
                       int h, int w, uint8_t* frame) {
  orc_env_frame(seed, env, step, tag, h, w, frame);
  for (size_t i = 0; i < (size_t)h * w * 4; ++i) frame[i] &= 63;
  int band = h / n_actions, g = (int)orc_pattern_goal(seed, env, step, n_actions);
  for (int y = band * g; y < band * (g + 1); ++y)
    memset(frame + (size_t)y * w * 4, 255, (size_t)w * 4);
}
void orc_pattern_reset(uint64_t seed, int n_e, int n_actions, int h, int w, uint8_t* frames) {
  for (int e = 0; e < n_e; ++e)
    orc_pattern_frame(seed, (uint32_t)e, 0u, 0u, n_actions, h, w, frames + (size_t)e * h * w * 4);
}
void orc_pattern_step(uint64_t seed, int n_e, uint32_t step, const int32_t* actions, uint32_t term_denom, int n_actions,
                      int h, int w, uint8_t* next_frames, int8_t* rewards, uint8_t* terminals,
                      int32_t* ep_len, int32_t* ep_return, int32_t* episodes) {
#pragma omp parallel for schedule(static)
  for (int e = 0; e < n_e; ++e) {
    int8_t unused;
    orc_env_outcome(seed, (uint32_t)e, step, actions[e], term_denom, &unused, &terminals[e]);
    rewards[e] = (uint32_t)actions[e] == orc_pattern_goal(seed, (uint32_t)e, step, n_actions) ? 1 : 0;
    uint32_t tag = terminals[e] ? 0u : (uint32_t)actions[e] + 1u;
    orc_pattern_frame(seed, (uint32_t)e, step + 1u, tag, n_actions, h, w, next_frames + (size_t)e * h * w * 4);
    ep_len[e] += 1; ep_return[e] += rewards[e];
    if (terminals[e]) { episodes[e] += 1; ep_len[e] = 0; ep_return[e] = 0; }
  }
}

/* ------------------------------------------------------------------ */
/* Forward pass f(s; theta) -> (logits, V)  (Section 5.1: one CNN, a     */
/* softmax policy head and a linear scalar value head)                  */
/* act[l]: float [n][h][w][c] of conv layer l (post ReLU), act[n_conv]: */
/* float [n][fc].  Pixels enter as integers; the 1/255 normalisation is */
/* applied to the finished sum of the first layer.                      */
/* ------------------------------------------------------------------ */
void orc_forward(const orc_net* net, const float* theta, int bf16, const uint8_t* frames, int n,
                 float** act, float* logits /* [n][A] */, float* values /* [n] */) {
  for (int l = 0; l < net->n_conv; ++l) {
    int H, W, C; layer_in_shape(net, l, &H, &W, &C);
    int K = net->k[l], S = net->stride[l], CO = net->cout[l];
    int OH = conv_out(H, K, S), OW = conv_out(W, K, S);
    const float* Wt = theta + off_conv_w(net, l);
    const float* bias = Wt + conv_w_size(net, l);
    const double scale = (l == 0) ? 1.0 / 255.0 : 1.0;
#pragma omp parallel for schedule(static)
    for (int b = 0; b < n; ++b)
      for (int oh = 0; oh < OH; ++oh)
        for (int ow = 0; ow < OW; ++ow)
          for (int co = 0; co < CO; ++co) {
            double acc = 0.0;
            for (int r = 0; r < K; ++r)
              for (int s = 0; s < K; ++s)
                for (int ci = 0; ci < C; ++ci) {
                  size_t ii = (((size_t)b * H + (oh * S + r)) * W + (ow * S + s)) * C + ci;
                  double x = (l == 0) ? (double)frames[ii] : (double)act[l - 1][ii];
                  double wv = (double)rnd(Wt[(((size_t)co * K + r) * K + s) * C + ci], bf16);
                  acc += wv * x;
                }
            float z = (float)(acc * scale + (double)bias[co]);
            act[l][(((size_t)b * OH + oh) * OW + ow) * CO + co] = rnd(z > 0.f ? z : 0.f, bf16);
          }
  }
  {
    const size_t IN = fc_in(net); const int F = net->fc, L = net->n_conv;
    const float* Wt = theta + off_fc_w(net); const float* bias = Wt + IN * F;
    /* a net with no conv layer feeds normalised pixels straight to the fc layer */
    const double scale = (L == 0) ? 1.0 / 255.0 : 1.0;
#pragma omp parallel for schedule(static)
    for (int b = 0; b < n; ++b)
      for (int o = 0; o < F; ++o) {
        double acc = 0.0;
        for (size_t i = 0; i < IN; ++i) {
          double x = (L == 0) ? (double)frames[(size_t)b * IN + i] : (double)act[L - 1][(size_t)b * IN + i];
          acc += (double)rnd(Wt[(size_t)o * IN + i], bf16) * x;
        }
        float z = (float)(acc * scale + (double)bias[o]);
        act[L][(size_t)b * F + o] = rnd(z > 0.f ? z : 0.f, bf16);
      }
  }
  {
    const int F = net->fc, A = net->n_actions, L = net->n_conv;
    const float* Wp = theta + off_pi_w(net); const float* bp = Wp + (size_t)A * F;
    const float* Wv = theta + off_v_w(net);  const float* bv = Wv + F;
#pragma omp parallel for schedule(static)
    for (int b = 0; b < n; ++b) {
      const float* h = act[L] + (size_t)b * F;
      for (int k = 0; k < A; ++k) {
        double acc = 0.0;
        for (int i = 0; i < F; ++i) acc += (double)rnd(Wp[(size_t)k * F + i], bf16) * (double)h[i];
        logits[(size_t)b * A + k] = (float)(acc + (double)bp[k]);
      }
      double acc = 0.0;
      for (int i = 0; i < F; ++i) acc += (double)rnd(Wv[i], bf16) * (double)h[i];
      values[b] = (float)(acc + (double)bv[0]);
    }
  }
}

/* ------------------------------------------------------------------ */
/* Frame pre-processing (Section 5.1): of the raw frames an action      */
/* repeated four times produces, the per-pixel maximum of the two       */
/* latest is kept, turned into one channel of pixel intensity, scaled   */
/* from 210 x 160 down to 84 x 84, and becomes the newest of the four   */
/* frames that make a state.  Readings where the paper is silent:       */
/*  - the maximum is taken per colour channel, before the intensity;    */
/*  - intensity = (77 R + 150 G + 29 B + 128) >> 8 (the 0.299 / 0.587 / */
/*    0.114 luminance weights in 8-bit fixed point, rounded);           */
/*  - scaling is the area average: output pixel (y, x) is the mean of   */
/*    the source over [2.5 y, 2.5 (y+1)) x [160 x / 84, 160 (x+1) / 84),*/
/*    every source pixel weighted by the area it shares with that box,  */
/*    rounded half up; in integers, with lengths in units of 1/84 of a  */
/*    source pixel, weights are overlap lengths and the total 210 * 160;*/
/*  - a state's channels are its four latest frames, oldest first; with */
/*    no previous state (after a reset) the new frame fills all four.   */
/* raw_*: [n][210][160][3] uint8; state_*: [n][84][84][4] uint8.        */
/* ------------------------------------------------------------------ */
static int overlap(int a0, int a1, int b0, int b1) {
  int lo = a0 > b0 ? a0 : b0, hi = a1 < b1 ? a1 : b1;
  return hi > lo ? hi - lo : 0;
}
void orc_preprocess(const uint8_t* raw_prev, const uint8_t* raw_last, const uint8_t* state_in /* nullable */,
                    uint8_t* state_out, int n) {
  enum { SH = 210, SW = 160, OH = 84, OW = 84 };
  uint8_t* grey = (uint8_t*)malloc((size_t)SH * SW);
  for (int e = 0; e < n; ++e) {
    const uint8_t* a = raw_prev + (size_t)e * SH * SW * 3;
    const uint8_t* b = raw_last + (size_t)e * SH * SW * 3;
    for (int p = 0; p < SH * SW; ++p) {
      int c[3];
      for (int k = 0; k < 3; ++k) c[k] = a[3 * p + k] > b[3 * p + k] ? a[3 * p + k] : b[3 * p + k];
      grey[p] = (uint8_t)((77 * c[0] + 150 * c[1] + 29 * c[2] + 128) >> 8);
    }
    for (int y = 0; y < OH; ++y)
      for (int x = 0; x < OW; ++x) {
        long long acc = 0;
        for (int r = 0; r < SH; ++r) {
          int wy = overlap(SH * y, SH * (y + 1), OH * r, OH * (r + 1));
          if (!wy) continue;
          for (int cidx = 0; cidx < SW; ++cidx) {
            int wx = overlap(SW * x, SW * (x + 1), OW * cidx, OW * (cidx + 1));
            if (wx) acc += (long long)wy * wx * grey[r * SW + cidx];
          }
        }
        uint8_t v = (uint8_t)((acc + (long long)SH * SW / 2) / ((long long)SH * SW));
        size_t o = (((size_t)e * OH + y) * OW + x) * 4;
        if (state_in) {
          uint8_t c1 = state_in[o + 1], c2 = state_in[o + 2], c3 = state_in[o + 3];
          state_out[o] = c1; state_out[o + 1] = c2; state_out[o + 2] = c3; state_out[o + 3] = v;
        } else {
          state_out[o] = state_out[o + 1] = state_out[o + 2] = state_out[o + 3] = v;
        }
      }
  }
  free(grey);
}

/* The stacking half of the above by itself (Section 5.1: a state is the */
/* stack of the four latest pre-processed frames): the newest frame      */
/* [n][84][84] joins the previous state [n][84][84][4], oldest first;    */
/* where restart[e] != 0 (nullable: no restarts) the environment has     */
/* begun a new episode and the new frame fills all four channels.        */
void orc_stack_push(const uint8_t* state_in, const uint8_t* newest, const uint8_t* restart /* nullable */,
                    uint8_t* state_out, int n) {
  enum { OH = 84, OW = 84 };
  for (int e = 0; e < n; ++e)
    for (int p = 0; p < OH * OW; ++p) {
      size_t o = ((size_t)e * OH * OW + p) * 4;
      uint8_t v = newest[(size_t)e * OH * OW + p];
      if (restart && restart[e]) {
        state_out[o] = state_out[o + 1] = state_out[o + 2] = state_out[o + 3] = v;
      } else {
        uint8_t c1 = state_in[o + 1], c2 = state_in[o + 2], c3 = state_in[o + 3];
        state_out[o] = c1; state_out[o + 1] = c2; state_out[o + 2] = c3; state_out[o + 3] = v;
      }
    }
}

/* ------------------------------------------------------------------ */
/* Softmax policy, entropy and inverse-CDF sampling (Algorithm 1:       */
/* "Sample a_t from pi(a_t | s_t; theta)")                              */
/* ------------------------------------------------------------------ */
void orc_softmax(const float* z, int A, float* p, float* logp, float* entropy) {
  double m = z[0];
  for (int k = 1; k < A; ++k) if (z[k] > m) m = z[k];
  double s = 0.0;
  for (int k = 0; k < A; ++k) s += exp((double)z[k] - m);
  double lse = m + log(s), H = 0.0;
  for (int k = 0; k < A; ++k) {
    double lp = (double)z[k] - lse, pk = exp(lp);
    logp[k] = (float)lp; p[k] = (float)pk;
    H -= pk * lp;
  }
  *entropy = (float)H;
}

/* smallest k with u < p_0 + ... + p_k (float running sum in index order), else A-1 */
int32_t orc_sample(const float* p, int A, float u) {
  float c = 0.f;
  for (int k = 0; k < A; ++k) { c += p[k]; if (u < c) return k; }
  return A - 1;
}

/* distance from u to the nearest CDF boundary: a GPU/oracle action mismatch is
 * tolerated only when this is tiny */
float orc_cdf_margin(const float* p, int A, float u) {
  float c = 0.f, best = 2.f;
  for (int k = 0; k < A; ++k) { c += p[k]; float d = fabsf(u - c); if (d < best) best = d; }
  return best;
}

/* ------------------------------------------------------------------ */
/* n-step returns (Algorithm 1: R_{tmax+1} bootstrap, then              */
/* R_t = r_t + gamma R_{t+1} going backwards), cut at every terminal    */
/* transition, and advantages R_t - v_t.  Arrays are [t][n_e].          */
/* ------------------------------------------------------------------ */
void orc_returns(int n_e, int t_max, float gamma, const int8_t* rewards, const uint8_t* terminals,
                 const float* values /* [t_max+1][n_e] */, float* R /* [t_max][n_e] */, float* adv) {
  for (int e = 0; e < n_e; ++e) {
    float next = values[(size_t)t_max * n_e + e];
    for (int t = t_max - 1; t >= 0; --t) {
      size_t i = (size_t)t * n_e + e;
      double keep = terminals[i] ? 0.0 : 1.0;
      next = (float)((double)rewards[i] + (double)gamma * keep * (double)next);
      R[i] = next;
      adv[i] = (float)((double)next - (double)values[i]);
    }
  }
}

/* ------------------------------------------------------------------ */
/* Loss over the batch of B experiences and its gradient at the heads   */
/* L = 1/B sum_i [ -adv_i log pi(a_i|s_i) - beta H_i + c_v (R_i-V_i)^2 ] */
/* (Eqs. 9-10 / Algorithm 1's d-theta lines as one minimised scalar;    */
/* adv and R are constants).  stats = {policy term, value term, mean H} */
/* ------------------------------------------------------------------ */
void orc_head_grad(int B, int A, float beta, float value_coef, const float* logits, const float* values,
                   const int32_t* actions, const float* R, const float* adv,
                   float* dz /* [B][A] */, float* dV /* [B] */, double stats[3]) {
  double pol = 0.0, val = 0.0, ent = 0.0;
  for (int i = 0; i < B; ++i) {
    const float* z = logits + (size_t)i * A;
    double m = z[0]; for (int k = 1; k < A; ++k) if (z[k] > m) m = z[k];
    double s = 0.0; for (int k = 0; k < A; ++k) s += exp((double)z[k] - m);
    double lse = m + log(s), H = 0.0;
    for (int k = 0; k < A; ++k) { double l = (double)z[k] - lse; H -= exp(l) * l; }
    for (int k = 0; k < A; ++k) {
      double l = (double)z[k] - lse, pk = exp(l);
      double g = -(double)adv[i] * ((k == actions[i] ? 1.0 : 0.0) - pk) + (double)beta * pk * (l + H);
      dz[(size_t)i * A + k] = (float)(g / B);
    }
    double d = (double)values[i] - (double)R[i];
    dV[i] = (float)(2.0 * (double)value_coef * d / B);
    pol += -(double)adv[i] * ((double)z[actions[i]] - lse);
    val += d * d; ent += H;
  }
  stats[0] = pol / B; stats[1] = (double)value_coef * val / B; stats[2] = ent / B;
}

/* ------------------------------------------------------------------ */
/* Value-based variant on the same framework (Section 3: the policy may */
/* be implicit; Section 2.2, Eqs. 2-4): the A outputs of the first head */
/* are Q(s, a; theta).  Acting is epsilon-greedy on Q; the target of    */
/* experience t is the n-step return bootstrapped from                  */
/* max_a' Q(s_{tmax+1}, a'; theta) (Eq. 3's target with the rewards of  */
/* the rollout in between, cut at terminals: orc_returns with that      */
/* bootstrap), and the loss is the batch mean of c (R_t - Q(s_t,a_t))^2 */
/* with R constant.  Eq. 4 prints the factor -1/2 where the derivative  */
/* of Eq. 3's square gives -2: the scale is the hyper-parameter c       */
/* (value_coef), as for the critic.                                     */
/* ------------------------------------------------------------------ */
/* arg max_a q[a], the smallest index among equals */
int32_t orc_q_greedy(const float* q, int A) {
  int best = 0;
  for (int k = 1; k < A; ++k) if (q[k] > q[best]) best = k;
  return best;
}
/* One uniform u in [0,1) decides both whether to explore and where: u < eps picks action
 * floor((u / eps) * A) (u / eps is uniform on [0,1) given u < eps), anything else is greedy.
 * The two float operations are single IEEE roundings, so any machine takes the same decision. */
int32_t orc_q_select(const float* q, int A, float u, float eps) {
  if (u < eps) {
    volatile float scaled = u / eps;
    volatile float pos = scaled * (float)A;
    int k = (int)pos;
    return k < A - 1 ? k : A - 1;
  }
  return orc_q_greedy(q, A);
}
/* gap between the largest and the second largest Q-value: a greedy mismatch between two
 * implementations is tolerated only when this is within their rounding */
float orc_q_margin(const float* q, int A) {
  int b = orc_q_greedy(q, A);
  float second = -INFINITY;
  for (int k = 0; k < A; ++k) if (k != b && q[k] > second) second = q[k];
  return q[b] - second;
}
/* L = (c / B) sum_i (R_i - Q_i[a_i])^2;  dL/dQ_i[k] = (2 c / B) (Q_i[a_i] - R_i) for k = a_i, else 0.
 * stats = {loss, mean of max_a Q} */
void orc_q_head_grad(int B, int A, float value_coef, const float* q, const int32_t* actions, const float* R,
                     float* dq /* [B][A] */, double stats[2]) {
  double loss = 0.0, qmax = 0.0;
  for (int i = 0; i < B; ++i) {
    const float* qi = q + (size_t)i * A;
    for (int k = 0; k < A; ++k) dq[(size_t)i * A + k] = 0.f;
    double d = (double)qi[actions[i]] - (double)R[i];
    dq[(size_t)i * A + actions[i]] = (float)(2.0 * (double)value_coef * d / B);
    loss += d * d;
    qmax += (double)qi[orc_q_greedy(qi, A)];
  }
  stats[0] = (double)value_coef * loss / B; stats[1] = qmax / B;
}

/* scalar loss in double with exact (unrounded) weights; used by the
 * finite-difference pin only */
double orc_loss_double(const orc_net* net, const double* theta, const uint8_t* frames, int n, float beta,
                       float value_coef, const int32_t* actions, const float* R, const float* adv) {
  size_t maxa = 0;
  for (int l = 0; l <= net->n_conv; ++l) if (orc_act_size(net, l) > maxa) maxa = orc_act_size(net, l);
  size_t in0 = (size_t)net->in_h * net->in_w * net->in_c; if (in0 > maxa) maxa = in0;
  double* buf0 = (double*)malloc(sizeof(double) * maxa);
  double* buf1 = (double*)malloc(sizeof(double) * maxa);
  double L = 0.0;
  for (int b = 0; b < n; ++b) {
    double* a = buf0; double* b2 = buf1;       /* a: layer input, b2: layer output */
    for (size_t i = 0; i < in0; ++i) a[i] = (double)frames[(size_t)b * in0 + i] / 255.0;
    size_t po = 0;
    for (int l = 0; l < net->n_conv; ++l) {
      int H, W, C; layer_in_shape(net, l, &H, &W, &C);
      int K = net->k[l], S = net->stride[l], CO = net->cout[l];
      int OH = conv_out(H, K, S), OW = conv_out(W, K, S);
      const double* Wt = theta + po; const double* bias = Wt + (size_t)CO * K * K * C;
      for (int oh = 0; oh < OH; ++oh) for (int ow = 0; ow < OW; ++ow) for (int co = 0; co < CO; ++co) {
        double acc = bias[co];
        for (int r = 0; r < K; ++r) for (int s = 0; s < K; ++s) for (int ci = 0; ci < C; ++ci)
          acc += Wt[(((size_t)co * K + r) * K + s) * C + ci] * a[((size_t)(oh * S + r) * W + (ow * S + s)) * C + ci];
        b2[((size_t)oh * OW + ow) * CO + co] = acc > 0 ? acc : 0;
      }
      po += (size_t)CO * K * K * C + CO;
      double* t = a; a = b2; b2 = t;
    }
    size_t IN = fc_in(net); int F = net->fc, A = net->n_actions;
    const double* Wt = theta + po; const double* bias = Wt + IN * F;
    for (int o = 0; o < F; ++o) {
      double acc = bias[o];
      for (size_t i = 0; i < IN; ++i) acc += Wt[(size_t)o * IN + i] * a[i];
      b2[o] = acc > 0 ? acc : 0;
    }
    po += IN * F + F;
    const double* Wp = theta + po; const double* bp = Wp + (size_t)A * F;
    const double* Wv = bp + A; const double* bv = Wv + F;
    double z[64], m = -1e300, s = 0, H = 0;
    for (int k = 0; k < A; ++k) {
      double acc = bp[k]; for (int i = 0; i < F; ++i) acc += Wp[(size_t)k * F + i] * b2[i];
      z[k] = acc; if (acc > m) m = acc;
    }
    for (int k = 0; k < A; ++k) s += exp(z[k] - m);
    double lse = m + log(s);
    for (int k = 0; k < A; ++k) H -= exp(z[k] - lse) * (z[k] - lse);
    double v = bv[0]; for (int i = 0; i < F; ++i) v += Wv[i] * b2[i];
    L += -(double)adv[b] * (z[actions[b]] - lse) - (double)beta * H
         + (double)value_coef * ((double)R[b] - v) * ((double)R[b] - v);
  }
  free(buf0); free(buf1);
  return L / n;
}

/* ------------------------------------------------------------------ */
/* Backward pass: from dL/dlogits, dL/dV to dL/dtheta by the chain rule. */
/* gact[l] (may be NULL entries): gradient w.r.t. the PRE-activation of */
/* layer l (ReLU mask already applied), float [n][...] as act[l].       */
/* Every sum runs in the fixed order (state, row, column) in double.    */
/* ------------------------------------------------------------------ */
void orc_backward(const orc_net* net, const float* theta, int bf16, const uint8_t* frames, int n,
                  float** act, const float* dz, const float* dV, float* grad, float** gact_out) {
  const int L = net->n_conv, F = net->fc, A = net->n_actions;
  const size_t IN = fc_in(net);
  memset(grad, 0, orc_param_count(net) * sizeof(float));
  float* gact[ORC_MAX_CONV + 1];
  for (int l = 0; l <= L; ++l) gact[l] = (float*)malloc(sizeof(float) * orc_act_size(net, l) * (size_t)n);

  /* heads */
  {
    const float* Wp = theta + off_pi_w(net); const float* Wv = theta + off_v_w(net);
    float* gWp = grad + off_pi_w(net); float* gbp = gWp + (size_t)A * F;
    float* gWv = grad + off_v_w(net);  float* gbv = gWv + F;
    const float* h = act[L];
#pragma omp parallel for schedule(static)
    for (int k = 0; k < A; ++k) {
      for (int i = 0; i < F; ++i) {
        double acc = 0.0;
        for (int b = 0; b < n; ++b) acc += (double)dz[(size_t)b * A + k] * (double)h[(size_t)b * F + i];
        gWp[(size_t)k * F + i] = (float)acc;
      }
      double acc = 0.0; for (int b = 0; b < n; ++b) acc += (double)dz[(size_t)b * A + k];
      gbp[k] = (float)acc;
    }
    for (int i = 0; i < F; ++i) {
      double acc = 0.0;
      for (int b = 0; b < n; ++b) acc += (double)dV[b] * (double)h[(size_t)b * F + i];
      gWv[i] = (float)acc;
    }
    { double acc = 0.0; for (int b = 0; b < n; ++b) acc += (double)dV[b]; gbv[0] = (float)acc; }
#pragma omp parallel for schedule(static)
    for (int b = 0; b < n; ++b)
      for (int i = 0; i < F; ++i) {
        double acc = 0.0;
        for (int k = 0; k < A; ++k) acc += (double)dz[(size_t)b * A + k] * (double)rnd(Wp[(size_t)k * F + i], bf16);
        acc += (double)dV[b] * (double)rnd(Wv[i], bf16);
        gact[L][(size_t)b * F + i] = h[(size_t)b * F + i] > 0.f ? rnd((float)acc, bf16) : 0.f;
      }
  }
  /* fully connected layer */
  {
    const float* Wt = theta + off_fc_w(net);
    float* gW = grad + off_fc_w(net); float* gb = gW + IN * F;
    const float* g = gact[L];
    const double scale = (L == 0) ? 1.0 / 255.0 : 1.0;
#pragma omp parallel for schedule(static)
    for (int o = 0; o < F; ++o) {
      double* acc = (double*)calloc(IN + 1, sizeof(double));
      for (int b = 0; b < n; ++b) {
        double go = (double)g[(size_t)b * F + o];
        acc[IN] += go;
        if (go == 0.0) continue;                       /* adds exact zeros otherwise */
        for (size_t i = 0; i < IN; ++i) {
          double x = (L == 0) ? (double)frames[(size_t)b * IN + i] : (double)act[L - 1][(size_t)b * IN + i];
          acc[i] += go * x;
        }
      }
      for (size_t i = 0; i < IN; ++i) gW[(size_t)o * IN + i] = (float)(acc[i] * scale);
      gb[o] = (float)acc[IN];
      free(acc);
    }
    if (L > 0) {
#pragma omp parallel for schedule(static)
      for (int b = 0; b < n; ++b)
        for (size_t i = 0; i < IN; ++i) {
          double acc = 0.0;
          for (int o = 0; o < F; ++o) acc += (double)g[(size_t)b * F + o] * (double)rnd(Wt[(size_t)o * IN + i], bf16);
          gact[L - 1][(size_t)b * IN + i] = act[L - 1][(size_t)b * IN + i] > 0.f ? rnd((float)acc, bf16) : 0.f;
        }
    }
  }
  /* conv layers, last to first */
  for (int l = L - 1; l >= 0; --l) {
    int H, W, C; layer_in_shape(net, l, &H, &W, &C);
    const int K = net->k[l], S = net->stride[l], CO = net->cout[l];
    const int OH = conv_out(H, K, S), OW = conv_out(W, K, S);
    const float* Wt = theta + off_conv_w(net, l);
    float* gW = grad + off_conv_w(net, l); float* gb = gW + conv_w_size(net, l);
    const float* g = gact[l];
    const double scale = (l == 0) ? 1.0 / 255.0 : 1.0;
    /* weight gradient: dW[co][r][s][ci] = sum_{b,oh,ow} g[b,oh,ow,co] * x[b, oh*S+r, ow*S+s, ci] */
#pragma omp parallel for schedule(dynamic, 1)
    for (int co = 0; co < CO; ++co) {
      const size_t wsz = (size_t)K * K * C;
      double* acc = (double*)calloc(wsz + 1, sizeof(double));
      for (int b = 0; b < n; ++b)
        for (int oh = 0; oh < OH; ++oh)
          for (int ow = 0; ow < OW; ++ow) {
            double go = (double)g[(((size_t)b * OH + oh) * OW + ow) * CO + co];
            acc[wsz] += go;
            if (go == 0.0) continue;
            for (int r = 0; r < K; ++r)
              for (int s = 0; s < K; ++s)
                for (int ci = 0; ci < C; ++ci) {
                  size_t ii = (((size_t)b * H + (oh * S + r)) * W + (ow * S + s)) * C + ci;
                  double x = (l == 0) ? (double)frames[ii] : (double)act[l - 1][ii];
                  acc[((size_t)r * K + s) * C + ci] += go * x;
                }
          }
      for (size_t i = 0; i < wsz; ++i) gW[(size_t)co * wsz + i] = (float)(acc[i] * scale);
      gb[co] = (float)acc[wsz];
      free(acc);
    }
    /* data gradient: d x[b,y,x,ci] = sum over the (r,s,co) whose window covers (y,x) */
    if (l > 0) {
#pragma omp parallel for schedule(static)
      for (int b = 0; b < n; ++b)
        for (int y = 0; y < H; ++y)
          for (int x = 0; x < W; ++x)
            for (int ci = 0; ci < C; ++ci) {
              double acc = 0.0;
              for (int r = 0; r < K; ++r) {
                int t = y - r; if (t < 0 || t % S) continue; int oh = t / S; if (oh >= OH) continue;
                for (int s = 0; s < K; ++s) {
                  int u = x - s; if (u < 0 || u % S) continue; int ow = u / S; if (ow >= OW) continue;
                  for (int co = 0; co < CO; ++co)
                    acc += (double)g[(((size_t)b * OH + oh) * OW + ow) * CO + co]
                         * (double)rnd(Wt[(((size_t)co * K + r) * K + s) * C + ci], bf16);
                }
              }
              size_t ii = (((size_t)b * H + y) * W + x) * C + ci;
              gact[l - 1][ii] = act[l - 1][ii] > 0.f ? rnd((float)acc, bf16) : 0.f;
            }
    }
  }
  for (int l = 0; l <= L; ++l) {
    if (gact_out && gact_out[l]) memcpy(gact_out[l], gact[l], sizeof(float) * orc_act_size(net, l) * (size_t)n);
    free(gact[l]);
  }
}

/* ------------------------------------------------------------------ */
/* Global-norm clipping (threshold c) followed by RMSProp               */
/* m <- rho m + (1-rho) g^2 ; theta <- theta - lr g / sqrt(m + eps)     */
/* returns 0, or 1 if the norm is not finite (then nothing is changed)  */
/* ------------------------------------------------------------------ */
int orc_clip_rmsprop(size_t P, float* theta, float* m, const float* grad, float lr, float rho, float eps,
                     float clip, double* norm_out, double* scale_out) {
  double ss = 0.0;
  for (size_t i = 0; i < P; ++i) ss += (double)grad[i] * (double)grad[i];
  double norm = sqrt(ss);
  *norm_out = norm;
  if (!isfinite(norm)) { *scale_out = 0.0; return 1; }
  double sc = (clip > 0.f && norm > (double)clip) ? (double)clip / norm : 1.0;
  *scale_out = sc;
  float scf = (float)sc;
  for (size_t i = 0; i < P; ++i) {
    double g = (double)scf * (double)grad[i];
    double mi = (double)rho * (double)m[i] + (1.0 - (double)rho) * g * g;
    m[i] = (float)mi;
    theta[i] = (float)((double)theta[i] - (double)lr * g / sqrt((double)m[i] + (double)eps));
  }
  return 0;
}
