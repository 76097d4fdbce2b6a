/*
 * kf_archive.h -- host-side bookkeeping for organising kernel variants and their measured results
 * the way the paper's search does (no GPU work; every pointer below is a HOST pointer).
 *
 * The paper keeps its candidate kernels in a MAP-Elites grid over three behavioural descriptors
 * with four levels each -- memory access pattern d_mem, algorithmic structure d_algo, parallelism
 * coordination d_sync, 4^3 = 64 cells (Section 3.2, "Kernel-Specific Behavioral Descriptors") --
 * one elite per cell, replaced only by a fitter child (Section 3.2, "MAP-Elites Algorithm").  It
 * records parent -> child transitions in a circular buffer and derives three gradient estimates per
 * cell from them: fitness gradient (Section 3.3, Eq. 1), improvement-rate gradient (Eq. 2) and
 * exploration gradient (Eq. 3), combined with weights 0.4 / 0.4 / 0.2.  This library has no language
 * model in the loop; it uses the same structures to file the variants its parameter sweep times
 * (python -m paper_2603_12440_b200.sweep) and to rank where the next variant should be tried.
 *
 * Readings where the paper gives no number: the time decay of Eq. 1 is
 * w(t) = 2^(-(now - iteration_t) / half_life); the set E of Eq. 3 is every empty cell (fitness 0)
 * plus every occupied cell whose fitness is below low_quality x the best fitness in the archive,
 * the cell itself excluded, and its proportionality constant is 1 / |E|; a conditional probability
 * over no transitions is 0.
 *
 * Ownership: kf_archive_create returns an object the caller destroys with kf_archive_destroy.
 * Calls on one object must not overlap in time.  Coordinates are int32[3], each in 0..3; anything
 * else is rejected (KF_ARCHIVE_BAD_ARG) and changes nothing.
 */
#ifndef KF_ARCHIVE_H
#define KF_ARCHIVE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kf_archive kf_archive;

enum {
    KF_ARCHIVE_IMPROVEMENT = 1, /* the child became the elite of its cell, or found an empty cell */
    KF_ARCHIVE_NEUTRAL = 0,     /* no archive update, fitness not below the parent's */
    KF_ARCHIVE_REGRESSION = -1, /* no archive update, fitness below the parent's */
    KF_ARCHIVE_BAD_ARG = -100
};

/* f(k) of Section 3.2, "Fitness Function": 0 if the variant does not compile, 0.1 if it compiles
 * but is incorrect, else 0.5 + 0.5 * min(1, speedup / target). */
double kf_fitness(int32_t compiled, int32_t correct, double speedup, double target);

/* ring_capacity: transitions kept (oldest dropped first), at least 1; half_life > 0 in iterations;
 * low_quality in [0, 1].  NULL on bad arguments or when memory runs out. */
kf_archive *kf_archive_create(int32_t ring_capacity, double half_life, double low_quality);
void kf_archive_destroy(kf_archive *a);

/* Offer a child.  It becomes the elite of cell `coords` if the cell is empty or its fitness is
 * higher than the incumbent's.  With parent_coords != NULL the transition (parent cell, child cell,
 * fitness - parent_fitness, outcome, iteration) is appended to the ring buffer.  Returns the
 * outcome. */
int32_t kf_archive_insert(kf_archive *a, const int32_t *coords, double fitness, int64_t id,
                          const int32_t *parent_coords, double parent_fitness, int64_t iteration);

/* 1 and the elite's fitness / id if the cell is occupied, 0 if empty, KF_ARCHIVE_BAD_ARG. */
int32_t kf_archive_cell(const kf_archive *a, const int32_t *coords, double *fitness, int64_t *id);

/* Transitions currently in the ring buffer. */
int32_t kf_archive_transitions(const kf_archive *a);

/* Gradient estimates for cell `coords` at iteration `now`: grad[3] = 0.4 F + 0.4 R + 0.2 E;
 * components[9] (may be NULL) = F[3], R[3], E[3].  Returns 0, or KF_ARCHIVE_BAD_ARG. */
int32_t kf_archive_gradient(const kf_archive *a, const int32_t *coords, int64_t now, double *grad,
                            double *components);

/* Selection weights of the occupied cells, proportional to exp(|grad|_2) and summing to 1
 * (Section 3.3, "Gradient-to-Prompt Translation": cells with strong gradients are sampled more).
 * coords_out[3 * 64], weights_out[64]; cells in row-major order of (d_mem, d_algo, d_sync).
 * Returns the number of occupied cells. */
int32_t kf_archive_sampling_weights(const kf_archive *a, int64_t now, int32_t *coords_out,
                                    double *weights_out);

#ifdef __cplusplus
}
#endif
#endif
