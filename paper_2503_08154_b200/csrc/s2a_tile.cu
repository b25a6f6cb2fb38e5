// Host side of the pipelined tile path: launch-shape policy, argument packing, the
// per-device error word.
#include "s2a_tile.cuh"

#include <stdio.h>
#include <stdlib.h>

#include <atomic>

namespace s2a {

__device__ unsigned int g_error_word = 0;

cudaError_t launch_tile_gelu_fwd(int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st);
cudaError_t launch_tile_gelu_bwd(int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st);
cudaError_t launch_tile_softmax_fwd(int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st);
cudaError_t launch_tile_softmax_bwd(int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st);
cudaError_t launch_tile_silu_fwd(int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st);
cudaError_t launch_tile_silu_bwd(int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st);
cudaError_t launch_tile_bits(int kernel, int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st);
cudaError_t launch_tile_pair_widths(int kernel, int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st);

namespace {

constexpr uint32_t kMaxStageBytes = 56 * 1024;   // tiles are not grown beyond this
constexpr uint32_t kHardStageBytes = 176 * 1024;  // the smallest legal tile may be this large (one CTA per SM,
                                                  // and a single stage beyond ~96 KB)

// Launch-shape overrides for tuning sweeps exist only in a library built with -DS2A_TUNING
// (build.py --tuning writes it to a file of its own).  The library proper reads no
// environment variable: a plan is a pure function of its arguments and the device.
#ifdef S2A_TUNING
// An override may be given for one kernel only: K<kernel id>_<name> (K3_S2A_CTAS_PER_SM=3) is
// looked up before <name>.
thread_local int tuning_kernel = -1;
int env_int(const char* name, int dflt) {
  char scoped[96];
  snprintf(scoped, sizeof scoped, "K%d_%s", tuning_kernel, name);
  const char* v = getenv(scoped);
  if (!(v && *v)) v = getenv(name);
  return (v && *v) ? atoi(v) : dflt;
}
const char* env_str(const char* name) { return getenv(name); }
#else
constexpr int env_int(const char*, int dflt) { return dflt; }
constexpr const char* env_str(const char*) { return nullptr; }
#endif

uint32_t gcd_u32(uint32_t a, uint32_t b) {
  while (b) { uint32_t t = a % b; a = b; b = t; }
  return a;
}

uint32_t align_up(uint32_t v, uint32_t a) { return (v + a - 1) / a * a; }

// SMs of the current device, looked up once per device.  Concurrent first calls may both
// query and store the same value.
int sm_count() {
  static std::atomic<int> cached[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return 148;  // no device visible (planning on a build host): assume a B200
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    cached[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

unsigned int* error_word_address() {
  // one address per device; looked up on first use with that device current (two threads
  // making the first call both store the same address)
  static std::atomic<unsigned int*> addr[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  unsigned int* a = addr[dev].load(std::memory_order_acquire);
  if (!a) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_error_word) != cudaSuccess) return nullptr;
    a = (unsigned int*)p;
    addr[dev].store(a, std::memory_order_release);
  }
  return a;
}

}  // namespace

// Launch-shape policy.  In a -DS2A_TUNING build (and only there) the environment overrides
// it: S2A_PATH=rowwise disables this path; S2A_UNIT, S2A_TILE_ROWS, S2A_WARPS, S2A_STAGES,
// S2A_CTAS_PER_SM, S2A_VARIANT=generic|any, S2A_FIXED=0, S2A_PDL=0, S2A_SPREAD=0,
// S2A_SINGLE_STAGE=0.
TilePlan plan_tile(int kernel, int dt, uint64_t n_rows, uint32_t L, int bits) {
  TilePlan p{};
  p.bits = (uint32_t)bits;
#ifdef S2A_TUNING
  tuning_kernel = kernel;
#endif
  if (bits != 4 && bits != 2 && bits != 8) return p;
  const char* path = env_str("S2A_PATH");
  if (path && path[0] == 'r') return p;
  const char* var = env_str("S2A_VARIANT");
  const bool force_generic = var && var[0] == 'g';
  const bool is_gelu = is_act_fwd(kernel) || is_act_bwd(kernel);  // GELU and SiLU share their kernels
  const bool is_silu = act_of(kernel) == 1;
  const uint32_t esize = dt == kF32 ? 4u : 2u;
  const uint32_t vec = 16u / esize;  // elements per 16-byte access
  // attention widths with fixed-length kernels of their own (ViT 197 / 257, DeiT 198, no class
  // token 196, patch-32 models 49 / 50, 145, and 577 / 1025 of the 384 / 512 pixel models): read as 2-element words even where 16-byte
  // vectors would fit (196 in binary32)
  const bool pair_width = !is_gelu && bits == 4 && !force_generic && !(var && var[0] == 'a') &&
                          (L == 197 || L == 257 || L == 49 || L == 50 || L == 145 || L == 196 || L == 198 || L == 577 ||
                           L == 1025);
  const bool vec16 = (L % vec) == 0 && !pair_width && !(bits != 4 && !is_gelu && (L == 197 || L == 257));
  const uint32_t epa = vec16 ? vec : 2u;
  const uint32_t n_acc = vec16 ? L / vec : (L + 1) / 2;  // accesses covering one row
  // rows per tile: the tile's code bytes must be a multiple of 16 (its element count a
  // multiple of 32 at 4 bits), its row count even
  const uint32_t epc = 128u / (uint32_t)bits;  // elements per 16 code bytes
  uint32_t r_min = epc / gcd_u32(L, epc);
  if (r_min < 2) r_min = 2;
  // Widths 577 and 1025: only every 32nd row starts on a 16-byte boundary of the code tensor, and
  // 32 rows are 37-131 KB of data: two stages at best, a single one for binary32 rows of 1025.
  // Their kernels can take tiles whose codes start anywhere (see tile_kernel's RAGGED): the row
  // count only has to make the DATA a multiple of 16 bytes (and be even), so a tile is 8 or 16
  // rows.  Measured on [97536, 1025] and [173280, 577], forward / backward TB/s, aligned 32-row
  // tiles -> ragged ones: 1025 binary32 3.27 / 5.24 -> 5.62 / 6.25, 1025 bfloat16 5.54 / 6.15 ->
  // 6.00 / 5.6, 577 binary32 5.78 / 5.87 -> 6.09 / 6.72, 577 bfloat16 5.81 / 5.59 -> 5.7 / 5.91:
  // taken wherever it won.
  const bool sm_fwd = kernel == kSoftmaxFwd, sm_bwd = kernel == kSoftmaxBwd;
  const bool ragged = pair_width && env_int("S2A_RAGGED", 1) != 0 &&
                      ((L == 1025 && !(dt == kBF16 && sm_bwd)) || (L == 577 && !(dt == kBF16 && sm_fwd)));
  if (ragged) {
    r_min = 16u / gcd_u32(L * esize, 16u);
    if (r_min < 2) r_min = 2;
  }
  if ((uint64_t)r_min * L * esize > kHardStageBytes) return p;

  uint32_t variant = kVariantGeneric, unit = 0, iters = 0;
  const int env_unit = env_int("S2A_UNIT", 0);
  const bool pair_bits = bits != 4 && !is_gelu && !force_generic && !(var && var[0] == 'a') && (L == 197 || L == 257);
  if (pair_bits) {
    // other code widths at the ViT attention widths: fixed-width kernels of their own (8 bits:
    // a byte per element, nothing shared; 2 bits: unpacked scratch bytes, packed per tile)
    variant = kVariantPairFixed;
    unit = 8;
    iters = (n_acc + unit - 1) / unit;
  } else if (bits != 4 && (kernel == kSoftmaxFwd || kernel == kSoftmaxBwd)) {
    // other code widths, softmax: the any-length form (aligned vectors, masked row ends)
    if (L < 16) return p;
    variant = kVariantAny;
    const uint32_t nvr = (L + vec - 1) / vec + 1;
    unit = 2;
    while (unit < 32 && (nvr + unit - 1) / unit > 4) unit *= 2;  // measured at 197: 8 lanes beat 4 and 16
    if (env_unit == 2 || env_unit == 4 || env_unit == 8 || env_unit == 16 || env_unit == 32) unit = (uint32_t)env_unit;
  } else if (bits != 4) {
    // other code widths: GELU rows of whole vectors, long enough for a two-warp unit
    if (!(kernel == kGeluFwd || kernel == kGeluBwd) || !vec16 || n_acc < 128) return p;
    variant = kVariantStream;
    unit = (dt == kF32 && n_acc >= 512) ? 128u : 64u;
    if (env_unit == 64 || env_unit == 128) unit = (uint32_t)env_unit;
  } else if (vec16 && !force_generic && is_gelu) {
    // streamed: nothing held in registers; a warp per row unless the row is short
    variant = kVariantStream;
    unit = n_acc >= 256 ? 64u : (n_acc >= 32 ? 32u : (n_acc >= 16 ? 16u : 8u));
    if (dt == kF32 && n_acc >= 512) unit = 128;  // the same vectors per lane as bfloat16 with 64
    if (env_unit == 8 || env_unit == 16 || env_unit == 32 || env_unit == 64 || env_unit == 128) unit = (uint32_t)env_unit;
    // a fixed vector count per lane (3..6, 8 or 10) when the row length allows it
    if (unit >= 64 && n_acc % unit == 0 && env_int("S2A_FIXED", 1) != 0) {
      const uint32_t per = n_acc / unit;
      if ((per >= 3 && per <= 6) || per == 8 || per == 10) iters = per;
    }
  } else if (vec16 && !force_generic) {
    // softmax on 16-byte vectors: up to 32 (at most 64) elements per lane in registers; rows
    // too long for a warp go to units of two or four warps
    const uint32_t cap = 32u / epa, cap2 = 64u / epa;
    const uint32_t units[5] = {8, 16, 32, 64, 128};
    for (int k = 0; k < 5 && unit == 0; ++k)
      if ((n_acc + units[k] - 1) / units[k] <= cap) unit = units[k];
    if (unit == 0 && (n_acc + 127) / 128 <= cap2) unit = 128;
    if (dt == kBF16 && n_acc > 4 && n_acc <= 8) unit = 4;  // 40..64 elements: two vectors per lane, one shuffle step less
    if (env_unit == 2 || env_unit == 4 || env_unit == 8 || env_unit == 16 || env_unit == 32 || env_unit == 64 ||
        env_unit == 128)
      unit = (uint32_t)env_unit;
    if (unit != 0 && (n_acc + unit - 1) / unit <= cap2) {
      variant = kVariantStream;
      iters = unit >= 64 ? 4 : (unit < 8 ? 2 : 1);
      while (iters < (n_acc + unit - 1) / unit) iters *= 2;
    } else {
      unit = 0;
    }
  } else if (pair_width) {
    variant = kVariantPairFixed;
    unit = L > 257 ? 32u : 8u;
    // the patch-32 widths: four lanes per row keep seven words each, so that the per-row
    // reductions and quotients weigh half as much against the per-element work
    if (L <= 50 && kernel == kSoftmaxFwd) unit = 4;
    if (env_unit == 4 || env_unit == 8) unit = (uint32_t)env_unit;
    iters = (n_acc + unit - 1) / unit;
  }
  const bool force_any = var && var[0] == 'a';
  if (!is_gelu && bits == 4 && !force_generic && L >= 16 &&
      (force_any || variant == kVariantGeneric || (variant == kVariantStream && unit == 0))) {
    // softmax rows of any other length (not whole vectors, or too long for registers):
    // aligned vectors with masked ends, streamed from shared memory.  A lane should walk
    // about 4 to 8 vectors per phase (measured: fewer and the row reductions dominate, more
    // and too few rows are in flight), so short rows get units of 1, 2 or 4 lanes.
    variant = kVariantAny;
    const uint32_t nvr = (L + vec - 1) / vec + 1;  // vectors a row can touch
    unit = 1;
    while (unit < 16 && (nvr + unit - 1) / unit > 8) unit *= 2;
    while (unit < 128 && (nvr + unit - 1) / unit > 16) unit *= 2;  // whole warps only for very long rows
    if (env_unit == 1 || env_unit == 2 || env_unit == 4 || env_unit == 8 || env_unit == 16 || env_unit == 32 ||
        env_unit == 64 || env_unit == 128)
      unit = (uint32_t)env_unit;
    iters = 0;
  }
  if (variant == kVariantGeneric && is_silu) return p;  // SiLU has the streamed form only
  if (variant == kVariantGeneric) {
    // general register-resident form: pair accesses with 8 or 32 lanes per row, or 16-byte
    // accesses with 128 lanes per row (long softmax rows)
    const uint32_t max_iters = (dt == kBF16 && vec16) ? 8u : 16u;
    if (vec16) {
      if (is_gelu) return p;
      unit = 128;
    } else {
      unit = (n_acc + 7) / 8 <= 16 ? 8u : 32u;
      if (env_unit == 8 || env_unit == 32) unit = (uint32_t)env_unit;
    }
    const uint32_t need = (n_acc + unit - 1) / unit;
    if (need > max_iters) return p;
    iters = 1;
    while (iters < need) iters *= 2;
  }

  uint32_t warps = unit == 128 ? 8u : 4u;
  if (variant == kVariantPairFixed && unit == 32) warps = 8;  // four row pairs in flight are too few (measured)
  // ragged tiles: 16 rows for eight warps, except (measured) binary32 1025 forward -- 8 rows, four
  // warps, two CTAs of two stages -- and binary32 577 backward -- 8 rows, four warps, one CTA of four stages
  const bool ragged_small = ragged && dt == kF32 && ((L == 1025 && sm_fwd) || (L == 577 && sm_bwd));
  if (ragged_small) warps = 4;
  if (variant == kVariantAny) {
    // eight consumer warps, four when that many sub-warp units would need a tile beyond 40 KB
    const uint32_t want = 256u / unit;  // rows that keep eight warps busy
    warps = (want > r_min && (uint64_t)want * L * esize > 40 * 1024) ? 4u : 8u;
  }
  if (variant == kVariantStream && !is_gelu) {
    // A softmax row is a chain of dependent phases (reduce, evaluate, reduce, ...).  With few
    // elements per lane, or the cheaper bfloat16 arithmetic, four warps leave the SM waiting
    // on shuffles; binary32 rows with 32 elements per lane run best with four, except the
    // one-warp units of 1024-element rows (measured at 512, 1024, 2048 and 4096).
    warps = (dt == kBF16 || iters * epa <= 16 || unit == 32) ? 8u : 4u;
    // The bfloat16 backward is light enough for four warps wherever a row is not exactly a warp's
    // (measured with the L2 prefetch in place, 4 against 8 warps: 128: 6.0 / 5.5 TB/s, 256: 6.2 / 5.6,
    // 512: 6.2 / 5.5, 2048: 6.5 / 5.8, 4096: 6.5 / 5.8; 1024, one warp per row: 5.7 / 6.2).
    if (dt == kBF16 && kernel == kSoftmaxBwd && unit >= 8 && unit != 32) warps = 4;
  }
  // bfloat16 rows of 40..64 elements (four lanes per row): four CTAs of four warps on 7-12 KB tiles
  // (64: forward 4.9 -> 5.1 TB/s, backward 5.8 -> 6.2)
  const bool short_rows = variant == kVariantStream && !is_gelu && dt == kBF16 && unit == 4 && bits == 4;
  if (short_rows) warps = 4;
  int ctas_per_sm = short_rows ? 4 : 2;
  if (variant == kVariantStream && is_gelu) ctas_per_sm = 4;
  if (variant == kVariantPairFixed) ctas_per_sm = 4;
  if (ragged_small && L == 577) ctas_per_sm = 1;
  // The GELU backward runs with eight warps on four-row tiles, two CTAs per SM: alone it gains
  // 1-3 % (hidden 4096 / 5120, where two rows leave room for two stages only), and in training
  // order, alternating with the softmax backward, the step gains 3 % (ViT-B/16 5733 -> 5917 GB/s,
  // L/16 5392 -> 5559, H/14 5463 -> 5593): most of what that alternation used to cost.
  // The forward takes the same shape only where two rows leave room for just two stages in a quarter
  // of the shared memory (hidden 4096 / 5120): alone it is then a little slower (5.78 -> 5.53 TB/s at
  // 4096), but alternating with the softmax forward the pair stops losing 4 us per launch (ViT-L/16
  // step 5598 -> 5727 GB/s; H/14 unchanged); at hidden 3072 (three stages) it measured slower both
  // ways, and so did this shape for either softmax kernel.
  const int shape_bits = env_int("S2A_X2", 1);  // tuning: bit 0 backward, bit 1 forward always, bit 4 forward never
  const bool two_stage_rows = (uint64_t)2 * L * esize * 5 / 4 > 17 * 1024;
  const bool wide_rows = variant == kVariantStream && is_gelu && bits == 4 && unit == 64 &&
                         ((is_act_bwd(kernel) && (shape_bits & 1)) ||
                          (is_act_fwd(kernel) && ((shape_bits & 2) || (two_stage_rows && (shape_bits & 16) == 0))));
  if (wide_rows) { warps = 8; ctas_per_sm = 2; }
  // one row at a time per unit; 2 bits: 64-row tiles (whole 16-byte code spans), eight warps, two
  // CTAs per SM; 8 bits: measured best with the 4-bit kernels' shape (5.2 against 4.9 TB/s)
  if (pair_bits && bits == 2) { warps = 8; ctas_per_sm = 2; }
  warps = (uint32_t)env_int("S2A_WARPS", (int)warps);
  if (warps < 1 || warps > 16 || (warps * 32) % unit != 0) return p;
  const uint32_t n_units = warps * 32 / unit;
  uint32_t G = (!vec16 && (L & 1u)) ? 2u : 1u;  // rows a unit takes per round
  if (variant == kVariantPairFixed) G = 2;       // always a pair, whatever the parity
  if (variant == kVariantAny) G = 1;              // shared code bytes are merged atomically
  if (variant == kVariantStream && kernel == kSoftmaxFwd) {
    const uint32_t held = iters * epa;            // elements a lane keeps per row
    G = held <= 8 ? 4u : (held <= 16 ? 2u : 1u);  // as StreamSoftmaxFwd::RPU
  }

  // tile rows: a multiple of r_min that gives every unit a row (pair) per round, within
  // the stage budget; prefer ~16 KiB of data per tile
  uint32_t rows = r_min;
  const uint32_t want_rows = n_units * G;
  while (rows % want_rows != 0 && (uint64_t)(rows + r_min) * L * esize <= kMaxStageBytes) rows += r_min;
  while ((uint64_t)rows * L * esize < 16 * 1024 && (uint64_t)rows * 2 * L * esize <= kMaxStageBytes) rows *= 2;
  if ((variant == kVariantStream && is_gelu) || variant == kVariantPairFixed || short_rows) {
    rows = r_min;  // small tiles: more CTAs per SM, each with its own pipeline
    while (rows % (n_units * G) != 0 && (uint64_t)(rows + r_min) * L * esize <= kMaxStageBytes) rows += r_min;
    if (short_rows)
      while ((uint64_t)rows * L * esize < 7 * 1024) rows *= 2;
    if (ragged) rows = n_units * G;  // one row pair per unit and round: 8 or 16 rows, multiples of r_min
  }
  rows = (uint32_t)env_int("S2A_TILE_ROWS", (int)rows);
  if (rows == 0 || rows % r_min != 0 || rows % G != 0 || (uint64_t)rows * L * esize > kHardStageBytes) return p;

  const uint32_t data_bytes = rows * L * esize;
  const uint32_t code_bytes = (uint32_t)((uint64_t)rows * L * (uint32_t)bits / 8);
  const uint32_t meta_bytes = rows * 8;
  const uint32_t code_off = align_up(data_bytes, 128);
  const uint32_t meta_off = code_off + align_up(code_bytes + (ragged ? 32u : 0u), 128);
  const uint32_t stage_bytes = meta_off + align_up(meta_bytes, 128);

  // CTAs per SM and stages per CTA.  Every tile kernel asks for a power-of-two fraction
  // of an SM's shared memory (1/4, 1/2 or all of it) and always for the WHOLE fraction:
  // with programmatic dependent launch the next kernel's CTAs move into the slots that
  // this kernel's CTAs leave, which only works smoothly when the slots have equal sizes
  // (measured: 50.5 KB and 52.5 KB requests in alternation cost 3.7 us per launch).
  // The fixed-width softmax backward with a tile too large for three stages in a quarter of the
  // shared memory (width 257: 20.9 KB stages) takes a third of it: three CTAs of three stages
  // measured 2.5 % faster than four of two (the forward, and width 197, measured slower that way).
  if (variant == kVariantPairFixed && kernel == kSoftmaxBwd && bits == 4 && ctas_per_sm == 4 &&
      (kMaxSmem / 4 - 1024 - kHeaderBytes) / stage_bytes < 3 && (kMaxSmem / 3 - 1024 - kHeaderBytes) / stage_bytes >= 3)
    ctas_per_sm = 3;
  ctas_per_sm = env_int("S2A_CTAS_PER_SM", ctas_per_sm);
  if (ctas_per_sm < 1 || ctas_per_sm > 4) ctas_per_sm = 2;
  {
    // registers bound the residency too: the kernels' register caps, by variant
    uint32_t regs = 128;
    if (variant == kVariantStream) regs = is_gelu ? 64u : (uint32_t)softmax_stream_regs(dt, (int)(iters * epa));
    if (variant == kVariantPairFixed) regs = 96;
    // the bfloat16 kernels at width 257 are built for 128 registers: three CTAs per SM
    if (variant == kVariantPairFixed && bits == 4 && dt == kBF16 && L == 257) {
      regs = 128;
      if (ctas_per_sm > 3) ctas_per_sm = 3;
    }
    if (variant == kVariantAny) regs = 80;
    while (ctas_per_sm > 1 && (uint64_t)regs * (warps + 1) * 32 * (uint32_t)ctas_per_sm > 65536) ctas_per_sm /= 2;
  }
  // beyond the stages: 256-entry derivative tables per unit (8-bit GELU backward), or the CTA's
  // scratch of the 2-bit fixed-width softmax forward: one unpacked code byte per element of a tile
  // (binary32), one byte per 2-element word (bfloat16)
  const uint32_t extra_bytes = (bits == 8 && is_gelu) ? n_units * 1024u
                               : ((pair_bits && bits == 2 && kernel == kSoftmaxFwd)
                                      ? align_up(dt == kBF16 ? rows * L / 2 : rows * L, 128) : 0u);
  const int env_stages = env_int("S2A_STAGES", 0);
  uint32_t stages = 0, smem = 0;
  for (int c = ctas_per_sm; c >= 1 && stages == 0; c = (c == 3 ? 2 : c / 2)) {
    const uint32_t budget = kMaxSmem / (uint32_t)c - 1024;  // 1 KiB per CTA is the system's
    const uint32_t fixed = kHeaderBytes + extra_bytes;
    uint32_t fit = budget > fixed ? (budget - fixed) / stage_bytes : 0;
    if (fit > 4) fit = 4;
    if (env_stages > 0 && (uint32_t)env_stages <= fit) fit = (uint32_t)env_stages;
    if (fit >= 2) { stages = fit; ctas_per_sm = c; smem = budget; }
  }
  if (stages == 0 && env_int("S2A_SINGLE_STAGE", 1) != 0) {
    // A tile too large to double-buffer: one CTA per SM with a single stage.  Load, row work
    // and store of a CTA then run one after the other, but the SMs drift out of step and
    // keep the memory system busy between them -- still well ahead of the row-at-a-time path.
    const uint32_t budget = kMaxSmem - 1024;
    const uint32_t fixed = kHeaderBytes + extra_bytes;
    if (budget > fixed && stage_bytes <= budget - fixed) { stages = 1; ctas_per_sm = 1; smem = budget; }
  }
  if (stages == 0) return p;

  p.n_tiles = n_rows / rows;
  // the backward loads the aligned span that covers a tile's codes: where that span of the very
  // last tile would reach beyond the code tensor, that tile is left to the row-at-a-time path
  if (ragged && p.n_tiles != 0 && n_rows % rows == 0 && (p.n_tiles * code_bytes) % 16 != 0) p.n_tiles -= 1;
  p.ragged_codes = ragged ? 1u : 0u;
  if (p.n_tiles == 0) return TilePlan{};
  p.tile_rows = rows;
  p.variant = variant;
  p.unit_lanes = unit;
  p.vec_elems = epa;
  p.iters = iters;
  p.warps = warps;
  p.stages = stages;
  p.smem_bytes = smem;
  uint64_t grid = (uint64_t)sm_count() * (uint32_t)ctas_per_sm;
  if (grid > p.n_tiles) grid = p.n_tiles;
  p.grid = (uint32_t)grid;
  p.overlap_launch = env_int("S2A_PDL", 1) != 0 ? 1u : 0u;
  p.rows_per_group = G;
  {
    // The sub-warp units of one warp may take row groups a fixed stride apart (different
    // shared-memory banks for the odd attention widths); that needs every unit of a warp to
    // find a group in every round, i.e. the tile's groups to divide evenly among them.
    const uint32_t upw = unit < 32 ? 32 / unit : 1;
    const uint32_t n_groups = rows / G;
    p.spread_units = (upw > 1 && n_groups % upw == 0 && env_int("S2A_SPREAD", 1) != 0) ? 1u : 0u;
    if (pair_bits && bits == 2) p.spread_units = 0;  // a warp's units must hold consecutive row pairs
  }
  return p;
}

cudaError_t launch_tile(int kernel, int dt, const TilePlan& p, const TileArgs& a, cudaStream_t st) {
  TileKernelArgs ka;
  ka.in = (const unsigned char*)a.in;
  ka.out = (unsigned char*)a.out;
  ka.codes = a.codes;
  ka.meta = (unsigned char*)a.meta;
  ka.tiles_per_cta = a.n_tiles / p.grid;
  ka.tiles_extra = (uint32_t)(a.n_tiles % p.grid);
  ka.row_len = a.row_len;
  ka.tile_rows = p.tile_rows;
  const uint32_t esize = dt == kF32 ? 4u : 2u;
  ka.data_bytes = p.tile_rows * a.row_len * esize;
  ka.code_bytes = (uint32_t)((uint64_t)p.tile_rows * a.row_len * p.bits / 8);
  ka.meta_bytes = p.tile_rows * 8;
  ka.code_off = align_up(ka.data_bytes, 128);
  ka.meta_off = ka.code_off + align_up(ka.code_bytes + (p.ragged_codes ? 32u : 0u), 128);  // as plan_tile
  ka.stage_bytes = ka.meta_off + align_up(ka.meta_bytes, 128);
  ka.stages = p.stages;
  ka.tab_off = p.bits != 4 ? kHeaderBytes + p.stages * ka.stage_bytes : 0u;  // the area after the stages
  ka.spread_units = p.spread_units;
  // two tiles per CTA ahead of the dependency wait (measured on the ViT-B/16 step: 0 tiles
  // 5286 GB/s, 1: 5640, 2: 5810, 3: 5700, 4: 5666, 6: 5407 -- more than the first two compete
  // with the predecessor's last stores)
  ka.prefetch_tiles = p.overlap_launch ? (uint32_t)env_int("S2A_PREFETCH", p.stages < 2 ? (int)p.stages : 2) : 0u;
  ka.prefetch_ahead = (uint32_t)env_int("S2A_X1", 0);
  ka.ragged_codes = p.ragged_codes;
  ka.error_word = error_word_address();
  if (!ka.error_word) return cudaErrorInvalidDevice;
  if (p.bits != 4) return launch_tile_bits(kernel, dt, p, &ka, st);
  if (p.variant == kVariantPairFixed && a.row_len != 197 && a.row_len != 257)
    return launch_tile_pair_widths(kernel, dt, p, &ka, st);
  switch (kernel) {
    case kGeluFwd: return launch_tile_gelu_fwd(dt, p, &ka, st);
    case kGeluBwd: return launch_tile_gelu_bwd(dt, p, &ka, st);
    case kSoftmaxFwd: return launch_tile_softmax_fwd(dt, p, &ka, st);
    case kSoftmaxBwd: return launch_tile_softmax_bwd(dt, p, &ka, st);
    case kSiluFwd: return launch_tile_silu_fwd(dt, p, &ka, st);
    case kSiluBwd: return launch_tile_silu_bwd(dt, p, &ka, st);
  }
  return cudaErrorInvalidValue;
}

// One warp waits, with a 2 ms limit, for a barrier phase that nothing will ever complete: the
// give-up path of the bounded wait (record the bit, return) run on purpose, so that a test can
// see the error word change and the context stay usable.
namespace {
__global__ void wait_expiry_probe(unsigned int* error_word) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_barrier_init();
  }
  __syncthreads();
  mbar_wait(&bar, 0, error_word, kErrSelfTest, 2000000ull);
}
}  // namespace

cudaError_t launch_wait_expiry_probe(cudaStream_t st) {
  unsigned int* err = error_word_address();
  if (!err) return cudaErrorInvalidDevice;
  wait_expiry_probe<<<1, 32, 0, st>>>(err);
  return cudaGetLastError();
}

// The fixed-width bfloat16 softmax forward takes a row's smallest and largest y from its smallest
// and largest x.  That holds when every operation between x and y never decreases as its input
// grows: the correctly rounded ones (fused multiply-add, product, rounding to bfloat16) cannot;
// the hardware's approximate 2^x is CHECKED here, over every binary32 argument the kernel can hand
// it (-150 .. 1; below -126 the result is flushed to zero): neighbouring arguments are compared
// and the pairs out of order are counted.
namespace {
__device__ unsigned long long g_exp2_out_of_order;
constexpr uint32_t kBitsMinus150 = 0xC3160000u, kBitsMinusZero = 0x80000000u, kBitsOne = 0x3F800000u;
__global__ void exp2_monotone_probe() {
  const uint64_t n_neg = kBitsMinus150 - kBitsMinusZero, n_pos = kBitsOne;
  unsigned long long bad = 0;
  for (uint64_t k = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; k < n_neg + n_pos; k += (uint64_t)gridDim.x * blockDim.x) {
    if (k < n_neg) {  // negative arguments: the larger bit pattern is the smaller number
      const uint32_t b = kBitsMinusZero + (uint32_t)k;
      bad += ex2_approx(__uint_as_float(b + 1)) > ex2_approx(__uint_as_float(b));
    } else {
      const uint32_t b = (uint32_t)(k - n_neg);
      bad += ex2_approx(__uint_as_float(b + 1)) < ex2_approx(__uint_as_float(b));
    }
  }
  if (bad) atomicAdd(&g_exp2_out_of_order, bad);
}
}  // namespace

cudaError_t count_exp2_out_of_order(unsigned long long* count, cudaStream_t st) {
  const unsigned long long zero = 0;
  cudaError_t e = cudaMemcpyToSymbolAsync(g_exp2_out_of_order, &zero, sizeof(zero), 0, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return e;
  exp2_monotone_probe<<<sm_count() * 8, 256, 0, st>>>();
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  e = cudaMemcpyFromSymbolAsync(count, g_exp2_out_of_order, sizeof(*count), 0, cudaMemcpyDeviceToHost, st);
  if (e != cudaSuccess) return e;
  return cudaStreamSynchronize(st);
}

cudaError_t read_error_word(unsigned int* flags, bool clear) {
  cudaError_t e = cudaMemcpyFromSymbol(flags, g_error_word, sizeof(unsigned int));
  if (e != cudaSuccess) return e;
  if (clear) {
    unsigned int zero = 0;
    e = cudaMemcpyToSymbol(g_error_word, &zero, sizeof(unsigned int));
  }
  return e;
}

}  // namespace s2a
