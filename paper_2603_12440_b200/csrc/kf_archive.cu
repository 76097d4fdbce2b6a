// Host-side archive of kernel variants (kf_archive.h): MAP-Elites grid over (d_mem, d_algo, d_sync),
// ring buffer of parent -> child transitions, gradient estimates of Section 3.3 (Eq. 1-3).
// No device code; compiled with the rest of the library so that one shared object carries the ABI.
#include <cmath>
#include <cstdint>
#include <new>
#include <vector>

#include "../../include/kf_archive.h"

namespace {

constexpr int kBins = 4, kDims = 3, kCells = kBins * kBins * kBins;
constexpr double kAlpha = 0.4, kBeta = 0.4, kGamma = 0.2;

struct Transition {
    int8_t parent[kDims], child[kDims];
    int32_t outcome;
    double delta_f;
    int64_t iteration;
};

inline bool coords_ok(const int32_t* c) {
    if (!c) return false;
    for (int d = 0; d < kDims; ++d)
        if (c[d] < 0 || c[d] >= kBins) return false;
    return true;
}
inline int cell_index(const int32_t* c) { return (c[0] * kBins + c[1]) * kBins + c[2]; }

}  // namespace

struct kf_archive {
    bool occupied[kCells] = {};
    double fitness[kCells] = {};
    int64_t id[kCells] = {};
    std::vector<Transition> ring;      // circular once full
    size_t head = 0;                   // index of the oldest transition when the ring is full
    size_t capacity = 0;
    double half_life = 1.0, low_quality = 0.5;
};

extern "C" {

double kf_fitness(int32_t compiled, int32_t correct, double speedup, double target) {
    if (!compiled) return 0.0;
    if (!correct) return 0.1;
    const double s = speedup / target;
    return 0.5 + 0.5 * (s < 1.0 ? s : 1.0);
}

kf_archive* kf_archive_create(int32_t ring_capacity, double half_life, double low_quality) {
    if (ring_capacity < 1 || !(half_life > 0.0) || !(low_quality >= 0.0 && low_quality <= 1.0)) return nullptr;
    kf_archive* a = new (std::nothrow) kf_archive;
    if (!a) return nullptr;
    a->capacity = (size_t)ring_capacity;
    a->half_life = half_life;
    a->low_quality = low_quality;
    try {
        a->ring.reserve(a->capacity);
    } catch (...) {
        delete a;
        return nullptr;
    }
    return a;
}

void kf_archive_destroy(kf_archive* a) { delete a; }

int32_t kf_archive_insert(kf_archive* a, const int32_t* coords, double fitness, int64_t id,
                          const int32_t* parent_coords, double parent_fitness, int64_t iteration) {
    if (!a || !coords_ok(coords) || (parent_coords && !coords_ok(parent_coords))) return KF_ARCHIVE_BAD_ARG;
    const int c = cell_index(coords);
    const bool became_elite = !a->occupied[c] || fitness > a->fitness[c];
    if (became_elite) {
        a->occupied[c] = true;
        a->fitness[c] = fitness;
        a->id[c] = id;
    }
    if (!parent_coords) return became_elite ? KF_ARCHIVE_IMPROVEMENT : KF_ARCHIVE_NEUTRAL;
    Transition t;
    for (int d = 0; d < kDims; ++d) {
        t.parent[d] = (int8_t)parent_coords[d];
        t.child[d] = (int8_t)coords[d];
    }
    t.delta_f = fitness - parent_fitness;
    t.outcome = became_elite ? KF_ARCHIVE_IMPROVEMENT : (t.delta_f < 0.0 ? KF_ARCHIVE_REGRESSION : KF_ARCHIVE_NEUTRAL);
    t.iteration = iteration;
    if (a->ring.size() < a->capacity) {
        a->ring.push_back(t);
    } else {
        a->ring[a->head] = t;          // overwrite the oldest
        a->head = (a->head + 1) % a->capacity;
    }
    return t.outcome;
}

int32_t kf_archive_cell(const kf_archive* a, const int32_t* coords, double* fitness, int64_t* id) {
    if (!a || !coords_ok(coords)) return KF_ARCHIVE_BAD_ARG;
    const int c = cell_index(coords);
    if (!a->occupied[c]) return 0;
    if (fitness) *fitness = a->fitness[c];
    if (id) *id = a->id[c];
    return 1;
}

int32_t kf_archive_transitions(const kf_archive* a) { return a ? (int32_t)a->ring.size() : 0; }

int32_t kf_archive_gradient(const kf_archive* a, const int32_t* coords, int64_t now, double* grad, double* components) {
    if (!a || !coords_ok(coords) || !grad) return KF_ARCHIVE_BAD_ARG;
    double F[kDims] = {}, R[kDims] = {}, E[kDims] = {};

    // Eq. 1 and Eq. 2 over the transitions that start in this cell, oldest first
    size_t n_from = 0;
    double up_all[kDims] = {}, up_imp[kDims] = {}, dn_all[kDims] = {}, dn_imp[kDims] = {};
    const size_t n = a->ring.size();
    for (size_t i = 0; i < n; ++i) {
        const Transition& t = a->ring[(a->head + i) % n];
        bool from_here = true;
        for (int d = 0; d < kDims; ++d) from_here = from_here && t.parent[d] == coords[d];
        if (!from_here) continue;
        ++n_from;
        const double w = std::exp2(-(double)(now - t.iteration) / a->half_life);
        for (int d = 0; d < kDims; ++d) {
            const int step = t.child[d] - t.parent[d];
            const int sgn = (step > 0) - (step < 0);
            F[d] += t.delta_f * sgn * w;
            if (step > 0) { up_all[d] += 1; up_imp[d] += t.outcome == KF_ARCHIVE_IMPROVEMENT; }
            if (step < 0) { dn_all[d] += 1; dn_imp[d] += t.outcome == KF_ARCHIVE_IMPROVEMENT; }
        }
    }
    for (int d = 0; d < kDims; ++d) {
        if (n_from) F[d] /= (double)n_from;
        R[d] = (up_all[d] > 0 ? up_imp[d] / up_all[d] : 0.0) - (dn_all[d] > 0 ? dn_imp[d] / dn_all[d] : 0.0);
    }

    // Eq. 3 over empty cells and low-quality occupied cells
    double fmax = 0.0;
    bool any = false;
    for (int c = 0; c < kCells; ++c)
        if (a->occupied[c] && (!any || a->fitness[c] > fmax)) { fmax = a->fitness[c]; any = true; }
    size_t n_e = 0;
    for (int i = 0; i < kBins; ++i)
        for (int j = 0; j < kBins; ++j)
            for (int k = 0; k < kBins; ++k) {
                const int cc[kDims] = {i, j, k};
                if (i == coords[0] && j == coords[1] && k == coords[2]) continue;
                const int c = (i * kBins + j) * kBins + k;
                double fc;
                if (!a->occupied[c]) fc = 0.0;
                else if (a->fitness[c] < a->low_quality * fmax) fc = a->fitness[c];
                else continue;
                ++n_e;
                double dist = 0.0;
                for (int d = 0; d < kDims; ++d) dist += std::fabs((double)(cc[d] - coords[d]));
                for (int d = 0; d < kDims; ++d) E[d] += (fmax - fc) / dist * (double)(cc[d] - coords[d]) / dist;
            }
    for (int d = 0; d < kDims; ++d) {
        if (n_e) E[d] /= (double)n_e;
        grad[d] = kAlpha * F[d] + kBeta * R[d] + kGamma * E[d];
        if (components) {
            components[d] = F[d];
            components[kDims + d] = R[d];
            components[2 * kDims + d] = E[d];
        }
    }
    return 0;
}

int32_t kf_archive_sampling_weights(const kf_archive* a, int64_t now, int32_t* coords_out, double* weights_out) {
    if (!a || !coords_out || !weights_out) return KF_ARCHIVE_BAD_ARG;
    int32_t n = 0;
    double sum = 0.0;
    for (int i = 0; i < kBins; ++i)
        for (int j = 0; j < kBins; ++j)
            for (int k = 0; k < kBins; ++k) {
                const int32_t cc[kDims] = {i, j, k};
                if (!a->occupied[cell_index(cc)]) continue;
                double g[kDims];
                kf_archive_gradient(a, cc, now, g, nullptr);
                const double w = std::exp(std::sqrt(g[0] * g[0] + g[1] * g[1] + g[2] * g[2]));
                for (int d = 0; d < kDims; ++d) coords_out[3 * n + d] = cc[d];
                weights_out[n] = w;
                sum += w;
                ++n;
            }
    for (int32_t i = 0; i < n; ++i) weights_out[i] /= sum;
    return n;
}

}  // extern "C"
