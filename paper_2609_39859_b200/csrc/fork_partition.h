/*
 * Static partition of one step's work over a persistent grid.
 *
 * The live rows of a step (masked positions inside their sequence's active block) are cut into
 * units of FORK_CHUNK vocabulary entries; with R rows and C units per row there are U = R*C
 * units, numbered row-major.  CTA g of G owns the contiguous unit range
 *     [ floor(g*U/G), floor((g+1)*U/G) ),
 * (G is first cut down to min(G, U)), so every CTA streams the same number of bytes (+-1 unit)
 * whatever R is.  A CTA writes one
 * partial result ("part") per row it overlaps, into slot r+g: along the unit order either r or g
 * (or both) grows from one part to the next, so r+g is unique and smaller than R+G.
 */
#ifndef FORK_PARTITION_H
#define FORK_PARTITION_H

#include <stdint.h>

#ifdef __CUDACC__
#define FORK_HD __host__ __device__ __forceinline__
#else
#define FORK_HD static inline
#endif

#define FORK_CHUNK 2048          /* vocabulary entries per unit */
#define FORK_MAX_GRID 2048       /* upper bound on the persistent grid, sizes the part array */

/* Only min(G, ceil(U / min_units)) CTAs take part, so that every participating CTA owns at least
   one unit (the range starts are then strictly increasing and the CTAs overlapping a row are
   consecutive) and, when the step is small, at least min_units of them on average: a step of a few
   rows is latency-bound whatever the number of CTAs, and every CTA less is a part less to publish,
   count and merge at the end. */
FORK_HD int32_t fork_effective_grid(int64_t U, int32_t G, int32_t min_units) {
  if (min_units < 1) min_units = 1;
  const int64_t cap = (U + min_units - 1) / min_units;
  return (cap < (int64_t)G) ? (int32_t)(cap < 1 ? 1 : cap) : G;
}

FORK_HD int64_t fork_part_begin(int64_t U, int32_t G, int32_t g) {
  return (int64_t)(((uint64_t)g * (uint64_t)U) / (uint64_t)G);
}

/* the CTA whose range holds unit x (0 <= x < U): the largest g with floor(g*U/G) <= x */
FORK_HD int32_t fork_part_owner(int64_t U, int32_t G, int64_t x) {
  return (int32_t)((((uint64_t)(x + 1)) * (uint64_t)G - 1ULL) / (uint64_t)U);
}

/* number of CTAs that overlap row r, i.e. the number of parts the row is reduced from */
FORK_HD int32_t fork_row_parts(int64_t U, int32_t G, int32_t C, int64_t r) {
  return fork_part_owner(U, G, (r + 1) * C - 1) - fork_part_owner(U, G, r * C) + 1;
}

#endif
