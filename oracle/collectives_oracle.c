/*
 * TEST INFRASTRUCTURE ONLY -- the plain CPU oracle for the collectives executor.
 *
 * Each function is the textbook definition of one collective written as naive
 * loops over [rank][element]; floating-point sums are carried in fp64, int32 sums
 * wrap as uint32, copy-only collectives move bytes.  There is no chunking, no
 * schedule, no blocking and no code shared with the CUDA path or its host
 * orchestrator.  Only the tests, the smoke check and the benchmark's cpu_baseline
 * leg may call into this file.
 *
 * Definitions follow the paper's statement of the collective contracts
 * (Sec. 2, "Stable communication semantics", including the V variants whose partition sizes
 * are given at run time), its layouts (Sec. 3.1: packed,
 * scattered, transposed and their V variants), and its reduction rule
 * (Sec. 3.3, Eq. "rank-order": one accumulator per element, starting from zero,
 * adding rank 0, 1, ..., n-1).  The MoE dispatch/combine pair is the expert-
 * parallel use of AllToAllV that Table 2 names; its row order is this build's
 * reading (see orc_moe_dispatch).
 *
 * Parity pins: every function here is pinned by tests that do not call it twice:
 * closed forms on rank-coded integers, AllToAll applied twice = identity,
 * AllReduce = AllGather o ReduceScatter (Sec. 3.1 "Composing transformations"),
 * float special cases, and brute force on tiny sizes.
 *
 * dtype codes: 0 = bf16 (uint16 bits), 1 = fp32, 2 = int32, 3 = bytes.
 */
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_BF16 = 0, ORC_F32 = 1, ORC_I32 = 2, ORC_U8 = 3 };

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

static double load_as_f64(const void *buf, int dtype, size_t i) {
  if (dtype == ORC_BF16) {
    uint32_t bits = ((uint32_t)((const uint16_t *)buf)[i]) << 16;
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
  }
  return (double)((const float *)buf)[i];
}

/* AllGather: in_r holds m bytes; out_r[p*m + i] = in_p[i] for every r, p. */
int orc_allgather(int R, size_t m_bytes, const void *const *in, void *const *out) {
  for (int r = 0; r < R; ++r)
    for (int p = 0; p < R; ++p) {
      const uint8_t *s = (const uint8_t *)in[p];
      uint8_t *d = (uint8_t *)out[r] + (size_t)p * m_bytes;
#pragma omp parallel for schedule(static)
      for (size_t i = 0; i < m_bytes; ++i) d[i] = s[i];
    }
  return 0;
}

/* AllToAll: in_r holds R partitions of m bytes; out_r[p*m + i] = in_p[r*m + i]. */
int orc_alltoall(int R, size_t m_bytes, const void *const *in, void *const *out) {
  for (int r = 0; r < R; ++r)
    for (int p = 0; p < R; ++p) {
      const uint8_t *s = (const uint8_t *)in[p] + (size_t)r * m_bytes;
      uint8_t *d = (uint8_t *)out[r] + (size_t)p * m_bytes;
#pragma omp parallel for schedule(static)
      for (size_t i = 0; i < m_bytes; ++i) d[i] = s[i];
    }
  return 0;
}

/* AllToAllV: counts[p*R + r] = bytes p sends to r.  Sender p lays its partitions
 * out in destination order, receiver r lays what it gets out in source order:
 *   soff_p[r] = sum_{q<r} C[p][q],  roff_r[p] = sum_{q<p} C[q][r],
 *   out_r[roff_r[p] + i] = in_p[soff_p[r] + i],  i < C[p][r]. */
int orc_alltoallv(int R, const uint64_t *counts, const void *const *in, void *const *out) {
  for (int r = 0; r < R; ++r)
    for (int p = 0; p < R; ++p) {
      size_t soff = 0, roff = 0;
      for (int q = 0; q < r; ++q) soff += counts[(size_t)p * R + q];
      for (int q = 0; q < p; ++q) roff += counts[(size_t)q * R + r];
      const uint8_t *s = (const uint8_t *)in[p] + soff;
      uint8_t *d = (uint8_t *)out[r] + roff;
      size_t n = counts[(size_t)p * R + r];
#pragma omp parallel for schedule(static)
      for (size_t i = 0; i < n; ++i) d[i] = s[i];
    }
  return 0;
}

/* AllGatherV (packedV -> scatteredV): rank p contributes n[p] bytes; every rank's output is
 * the contributions in rank order: out_r[off_p + i] = in_p[i], off_p = sum_{q<p} n[q]. */
int orc_allgatherv(int R, const uint64_t *n_bytes, const void *const *in, void *const *out) {
  for (int r = 0; r < R; ++r) {
    size_t off = 0;
    for (int p = 0; p < R; ++p) {
      const uint8_t *s = (const uint8_t *)in[p];
      uint8_t *d = (uint8_t *)out[r] + off;
      for (size_t i = 0; i < n_bytes[p]; ++i) d[i] = s[i];
      off += n_bytes[p];
    }
  }
  return 0;
}

/* ReduceScatterV (scatteredV -> packedV): every rank holds T = sum n[k] elements cut into
 * partitions of n[k] elements; rank k receives out_k[i] = sum_p in_p[off_k + i], i < n[k]. */
int orc_reduce_scatterv_f64(int R, int dtype, const uint64_t *n_elems, const void *const *in, double *const *out) {
  if (dtype != ORC_BF16 && dtype != ORC_F32) return 1;
  size_t off = 0;
  for (int k = 0; k < R; ++k) {
    for (size_t i = 0; i < n_elems[k]; ++i) {
      double acc = 0.0;
      for (int p = 0; p < R; ++p) acc += load_as_f64(in[p], dtype, off + i);
      out[k][i] = acc;
    }
    off += n_elems[k];
  }
  return 0;
}

int orc_reduce_scatterv_i32(int R, const uint64_t *n_elems, const void *const *in, int32_t *const *out) {
  size_t off = 0;
  for (int k = 0; k < R; ++k) {
    for (size_t i = 0; i < n_elems[k]; ++i) {
      uint32_t acc = 0;
      for (int p = 0; p < R; ++p) acc += ((const uint32_t *)in[p])[off + i];
      out[k][i] = (int32_t)acc;
    }
    off += n_elems[k];
  }
  return 0;
}

/* ReduceScatter (float): in_r holds R*m elements; out_r[i] = sum_p in_p[r*m + i],
 * ascending p from zero, in fp64 (the reference the float tolerance is set against). */
int orc_reduce_scatter_f64(int R, int dtype, size_t m, const void *const *in, double *const *out) {
  if (dtype != ORC_BF16 && dtype != ORC_F32) return 1;
  for (int r = 0; r < R; ++r) {
    double *d = out[r];
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < m; ++i) {
      double acc = 0.0;
      for (int p = 0; p < R; ++p) acc += load_as_f64(in[p], dtype, (size_t)r * m + i);
      d[i] = acc;
    }
  }
  return 0;
}

/* ReduceScatter (int32): same with wrapping two's-complement sums. */
int orc_reduce_scatter_i32(int R, size_t m, const void *const *in, int32_t *const *out) {
  for (int r = 0; r < R; ++r) {
    int32_t *d = out[r];
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < m; ++i) {
      uint32_t acc = 0;
      for (int p = 0; p < R; ++p) acc += ((const uint32_t *)in[p])[(size_t)r * m + i];
      d[i] = (int32_t)acc;
    }
  }
  return 0;
}

/* AllReduce (float): in_r holds n elements; out_r[i] = sum_p in_p[i] for every r. */
int orc_allreduce_f64(int R, int dtype, size_t n, const void *const *in, double *const *out) {
  if (dtype != ORC_BF16 && dtype != ORC_F32) return 1;
  for (int r = 0; r < R; ++r) {
    double *d = out[r];
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; ++i) {
      double acc = 0.0;
      for (int p = 0; p < R; ++p) acc += load_as_f64(in[p], dtype, i);
      d[i] = acc;
    }
  }
  return 0;
}

int orc_allreduce_i32(int R, size_t n, const void *const *in, int32_t *const *out) {
  for (int r = 0; r < R; ++r) {
    int32_t *d = out[r];
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; ++i) {
      uint32_t acc = 0;
      for (int p = 0; p < R; ++p) acc += ((const uint32_t *)in[p])[i];
      d[i] = (int32_t)acc;
    }
  }
  return 0;
}

/*
 * MoE dispatch (expert-parallel AllToAllV of token rows; scatteredV -> transposedV).
 *
 * Rank p holds x_p[T][row_bytes] and idx_p[T][K] (K distinct experts per token).
 * Expert e lives on rank e / (E/R).  One row is sent per (token, slot) pair.  The
 * receive buffer of rank r is in source-rank order (the transposed layout); inside
 * the segment from source p rows are grouped by expert ascending and, inside one
 * expert, by token ascending.  So the row order at r is (p, e, t), written here as
 * exactly those nested loops.
 *
 * Outputs: recv[r] rows; meta[r][row] = {p, t, slot, e}; pos[p][t*K+j] = row index
 * in the destination rank's receive buffer; counts[p*R + r] = rows p -> r;
 * expert_counts[p*E + e] = rows p -> e.  Returns 2 if a receive buffer overflows.
 */
int orc_moe_dispatch(int R, int T, int E, int K, size_t row_bytes, size_t recv_capacity_rows,
                     const void *const *x, const int32_t *const *idx, void *const *recv,
                     int32_t *const *meta, int32_t *const *pos, int64_t *counts,
                     int64_t *expert_counts) {
  const int epr = E / R;
  if (epr * R != E) return 1;
  memset(counts, 0, sizeof(int64_t) * (size_t)R * R);
  memset(expert_counts, 0, sizeof(int64_t) * (size_t)R * E);
  for (int r = 0; r < R; ++r) {
    size_t row = 0;
    for (int p = 0; p < R; ++p)
      for (int e = r * epr; e < (r + 1) * epr; ++e)
        for (int t = 0; t < T; ++t)
          for (int j = 0; j < K; ++j) {
            if (idx[p][(size_t)t * K + j] != e) continue;
            if (row >= recv_capacity_rows) return 2;
            memcpy((uint8_t *)recv[r] + row * row_bytes,
                   (const uint8_t *)x[p] + (size_t)t * row_bytes, row_bytes);
            int32_t *m = meta[r] + row * 4;
            m[0] = p; m[1] = t; m[2] = j; m[3] = e;
            pos[p][(size_t)t * K + j] = (int32_t)row;
            counts[(size_t)p * R + r] += 1;
            expert_counts[(size_t)p * E + e] += 1;
            ++row;
          }
  }
  return 0;
}

/*
 * MoE combine: out_p[t][h] = sum_{j=0}^{K-1} g_p[t][j] * y[rank(e_j)][pos_p[t][j]][h],
 * ascending j, in fp64; y rows are bf16 in the layout dispatch produced.
 */
int orc_moe_combine_f64(int R, int T, int H, int E, int K, const void *const *y,
                        const int32_t *const *idx, const int32_t *const *pos,
                        const float *const *gates, double *const *out) {
  const int epr = E / R;
  if (epr * R != E) return 1;
  for (int p = 0; p < R; ++p) {
    double *o = out[p];
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t)
      for (int h = 0; h < H; ++h) {
        double acc = 0.0;
        for (int j = 0; j < K; ++j) {
          int e = idx[p][(size_t)t * K + j];
          int r = e / epr;
          size_t row = (size_t)pos[p][(size_t)t * K + j];
          acc += (double)gates[p][(size_t)t * K + j] * load_as_f64(y[r], ORC_BF16, row * (size_t)H + h);
        }
        o[(size_t)t * H + h] = acc;
      }
  }
  return 0;
}

/*
 * MoE dispatch / combine with per-rank deduplication (the variant used when several of a
 * token's experts live on the same rank: the token row crosses to that rank once).
 *
 * Dispatch: rank r receives ONE row for every (source p, token t) that selects at least one
 * expert on r, in (p, t) order.  meta[r][row] = {p, t, slot mask, r}: bit j of the mask is set
 * when slot j's expert lives on r.  pos[p][t*R + r] = row at rank r, or -1.
 * counts[p*R + r] = rows p -> r.  Returns 2 on receive overflow.
 *
 * Combine: each rank returns one row per received row (the expert layer has already applied
 * the gates and summed its local experts); out_p[t][h] = sum over r ascending with
 * pos[p][t*R+r] >= 0 of z_r[pos][h], in fp64.
 */
int orc_moe_dispatch_dedup(int R, int T, int E, int K, size_t row_bytes, size_t recv_capacity_rows,
                           const void *const *x, const int32_t *const *idx, void *const *recv,
                           int32_t *const *meta, int32_t *const *pos, int64_t *counts) {
  const int epr = E / R;
  if (epr * R != E || K > 32) return 1;
  memset(counts, 0, sizeof(int64_t) * (size_t)R * R);
  for (int r = 0; r < R; ++r) {
    size_t row = 0;
    for (int p = 0; p < R; ++p)
      for (int t = 0; t < T; ++t) {
        uint32_t mask = 0;
        for (int j = 0; j < K; ++j)
          if (idx[p][(size_t)t * K + j] / epr == r) mask |= 1u << j;
        if (!mask) {
          pos[p][(size_t)t * R + r] = -1;
          continue;
        }
        if (row >= recv_capacity_rows) return 2;
        memcpy((uint8_t *)recv[r] + row * row_bytes, (const uint8_t *)x[p] + (size_t)t * row_bytes, row_bytes);
        int32_t *m = meta[r] + row * 4;
        m[0] = p; m[1] = t; m[2] = (int32_t)mask; m[3] = r;
        pos[p][(size_t)t * R + r] = (int32_t)row;
        counts[(size_t)p * R + r] += 1;
        ++row;
      }
  }
  return 0;
}

int orc_moe_combine_dedup_f64(int R, int T, int H, const void *const *z, const int32_t *const *pos,
                              double *const *out) {
  for (int p = 0; p < R; ++p)
    for (int t = 0; t < T; ++t)
      for (int h = 0; h < H; ++h) {
        double acc = 0.0;
        for (int r = 0; r < R; ++r) {
          int32_t row = pos[p][(size_t)t * R + r];
          if (row >= 0) acc += load_as_f64(z[r], ORC_BF16, (size_t)row * H + h);
        }
        out[p][(size_t)t * H + h] = acc;
      }
  return 0;
}
