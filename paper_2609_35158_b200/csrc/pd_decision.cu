// PD decision engine: the paper's closed-form makespan models and plan arithmetic as plain host functions.
//
// Eq. 1 (colocated makespan), Eq. 2-3 (disaggregated decode / prefill paths), the capacity constraints
// of Sec. 4.2, the enumeration over N_P with mode-dependent hysteresis (Sec. 4.3.2), the minimal-change
// counts of Eq. 5-6 with a concrete plan, and the toggle gate of Eq. 7. CPU only: these are O(workers)
// scalar formulas. They sit in this library because two of their inputs are measured by it: b, the
// per-sequence decode cost (the slope of the decode-attention step time over the number of concurrent
// sequences, pd_fit_decode_cost), and K, the KV bytes per token moved by pd_kv_gather / pd_kv_scatter.
#include "../../include/pd.h"

#include <cmath>
#include <cstring>

namespace {

bool valid_model(const pd_cost_model *m) {
    return m != nullptr && m->B > 0 && m->S > 0 && m->r >= 0 && m->dL >= 0 && m->theta >= 0 && m->A >= 0 && m->b >= 0 &&
           m->t_prefill >= 0 && m->T_over >= 0 && m->T_env >= 0 && m->K_bytes >= 0 && m->BW > 0 && m->K_seq_bytes >= 0 &&
           m->H_max_bytes > 0;
}

}  // namespace

extern "C" {

double pd_makespan_coloc(const pd_cost_model *m, int32_t N) {
    if (!valid_model(m) || N < 1) return NAN;
    // Eq. 1: T = S [ (B dL / N) t_prefill + r (A + b B / N) + T_over ] + T_env
    return m->S * ((m->B * m->dL / N) * m->t_prefill + m->r * (m->A + m->b * m->B / N) + m->T_over) + m->T_env;
}

double pd_makespan_disagg(const pd_cost_model *m, int32_t N_P, int32_t N_D, double *T_prefill, double *T_decode) {
    if (!valid_model(m) || N_P < 1 || N_D < 1) return NAN;
    // Eq. 2: T_decode = S r (A + b B / (N_D (1 + theta))) (1 + theta)
    const double td = m->S * m->r * (m->A + m->b * m->B / (N_D * (1.0 + m->theta))) * (1.0 + m->theta);
    // Eq. 3: T_prefill = S ( (B dL / N_P) t_prefill + B dL K / BW )
    const double tp = m->S * ((m->B * m->dL / N_P) * m->t_prefill + m->B * m->dL * m->K_bytes / m->BW);
    if (T_prefill != nullptr) *T_prefill = tp;
    if (T_decode != nullptr) *T_decode = td;
    return (tp > td ? tp : td) + m->T_env;  // T_dis = max(T_prefill, T_decode) + T_env
}

int32_t pd_feasible_disagg(const pd_cost_model *m, int32_t N_P, int32_t N_D) {
    if (!valid_model(m) || N_P < 1 || N_D < 1) return 0;
    // decode workers must hold the whole batch's KV cache: B K_seq <= N_D H_max
    if (m->B * m->K_seq_bytes > N_D * m->H_max_bytes) return 0;
    // prefill workers must absorb lambda_P = B S dL tokens per step; a capacity of 0 switches the check off
    if (m->prefill_tokens_per_worker > 0 && m->B * m->S * m->dL > N_P * m->prefill_tokens_per_worker) return 0;
    return 1;
}

int pd_decide(const pd_cost_model *m, int32_t N_k, const pd_target *current, double ratio_threshold,
              double mode_threshold, pd_target *out) {
    if (!valid_model(m) || N_k < 1 || out == nullptr || ratio_threshold < 0 || mode_threshold < 0)
        return PD_ERR_INVALID_ARG;
    // best candidate: colocation against every feasible split N_P in [1, N_k - 1]
    pd_target best{0, 0, N_k, pd_makespan_coloc(m, N_k)};
    for (int32_t np = 1; np <= N_k - 1; ++np) {
        const int32_t nd = N_k - np;
        if (!pd_feasible_disagg(m, np, nd)) continue;
        const double t = pd_makespan_disagg(m, np, nd, nullptr, nullptr);
        if (t < best.makespan) best = pd_target{np, nd, 0, t};
    }
    *out = best;
    if (current == nullptr) return PD_OK;
    // Is the current configuration still realisable with N_k workers? If not the switch is forced.
    const bool cur_coloc = current->N_C > 0;
    const int32_t cur_total = current->N_P + current->N_D + current->N_C;
    const bool cur_ok = cur_total == N_k && (cur_coloc ? (current->N_P == 0 && current->N_D == 0)
                                                       : pd_feasible_disagg(m, current->N_P, current->N_D) != 0);
    if (!cur_ok) return PD_OK;
    const double t_cur = cur_coloc ? pd_makespan_coloc(m, N_k) : pd_makespan_disagg(m, current->N_P, current->N_D, nullptr, nullptr);
    // Hysteresis: an alternative is admitted only if it beats the current makespan by more than its threshold
    // (a fraction of the current makespan, strictly) -- mode_threshold for a colocation <-> disaggregation
    // switch, ratio_threshold for another ratio of the same mode. The best admitted alternative wins, so a
    // refused mode switch does not block a ratio adjustment that clears the smaller threshold.
    pd_target choice{current->N_P, current->N_D, current->N_C, t_cur};
    auto consider = [&](const pd_target &c) {
        if (c.N_P == current->N_P && c.N_D == current->N_D && c.N_C == current->N_C) return;
        const double threshold = ((c.N_C > 0) != cur_coloc) ? mode_threshold : ratio_threshold;
        if (t_cur - c.makespan > threshold * t_cur && c.makespan < choice.makespan) choice = c;
    };
    consider(pd_target{0, 0, N_k, pd_makespan_coloc(m, N_k)});
    for (int32_t np = 1; np <= N_k - 1; ++np) {
        const int32_t nd = N_k - np;
        if (!pd_feasible_disagg(m, np, nd)) continue;
        consider(pd_target{np, nd, 0, pd_makespan_disagg(m, np, nd, nullptr, nullptr)});
    }
    *out = choice;
    return PD_OK;
}

int pd_min_change_plan(const int32_t *cur_active, const int32_t *cur_role, const int32_t *dst_active, int32_t n_slots,
                       const int32_t *dst_role_count, int32_t n_roles, int32_t *new_role, int32_t *d_worker,
                       int32_t *d_role) {
    if (cur_active == nullptr || cur_role == nullptr || dst_active == nullptr || dst_role_count == nullptr ||
        new_role == nullptr || n_slots < 0 || n_roles < 1 || n_roles > 16)
        return PD_ERR_INVALID_ARG;
    int32_t need[16], src[16];
    int32_t total_dst = 0, n_dst_active = 0, dw = 0;
    for (int r = 0; r < n_roles; ++r) {
        if (dst_role_count[r] < 0) return PD_ERR_INVALID_ARG;
        need[r] = dst_role_count[r];
        src[r] = 0;
        total_dst += dst_role_count[r];
    }
    for (int w = 0; w < n_slots; ++w) {
        const bool a = cur_active[w] != 0, d = dst_active[w] != 0;
        if (a && (cur_role[w] < 0 || cur_role[w] >= n_roles)) return PD_ERR_INVALID_ARG;
        n_dst_active += d;
        dw += a != d;  // Eq. 5: joins plus departures
        new_role[w] = -1;
    }
    if (n_dst_active != total_dst) return PD_ERR_INVALID_ARG;  // the target role counts must cover the target set
    // survivors keep their role up to the target count of that role
    for (int w = 0; w < n_slots; ++w) {
        if (!(cur_active[w] && dst_active[w])) continue;
        ++src[cur_role[w]];
        if (need[cur_role[w]] > 0) {
            new_role[w] = cur_role[w];
            --need[cur_role[w]];
        }
    }
    int32_t dr = 0;
    for (int r = 0; r < n_roles; ++r) {  // Eq. 6: sum over roles of n_src - min(n_src, n_dst)
        const int32_t keep = src[r] < dst_role_count[r] ? src[r] : dst_role_count[r];
        dr += src[r] - keep;
    }
    // the remaining deficits are filled by survivors that must switch, then by joining workers
    int r_fill = 0;
    auto next_deficit = [&]() {
        while (r_fill < n_roles && need[r_fill] == 0) ++r_fill;
        return r_fill;
    };
    for (int pass = 0; pass < 2; ++pass) {
        for (int w = 0; w < n_slots; ++w) {
            if (!dst_active[w] || new_role[w] >= 0) continue;
            const bool survivor = cur_active[w] != 0;
            if ((pass == 0) != survivor) continue;
            const int r = next_deficit();
            if (r >= n_roles) return PD_ERR_INVALID_ARG;
            new_role[w] = r;
            --need[r];
        }
    }
    if (d_worker != nullptr) *d_worker = dw;
    if (d_role != nullptr) *d_role = dr;
    return PD_OK;
}

int32_t pd_toggle_gate(double R, double B, double T_ded, double T_full, double T_toggle) {
    if (!(B > 0) || R < 0) return 0;
    return (R / B) * (T_ded - T_full) > T_toggle ? 1 : 0;  // Eq. 7
}

int pd_fit_decode_cost(const double *concurrency, const double *step_seconds, int32_t n, double *A, double *b) {
    if (concurrency == nullptr || step_seconds == nullptr || A == nullptr || b == nullptr || n < 2) return PD_ERR_INVALID_ARG;
    double sx = 0, sy = 0, sxx = 0, sxy = 0;
    for (int i = 0; i < n; ++i) {
        sx += concurrency[i];
        sy += step_seconds[i];
        sxx += concurrency[i] * concurrency[i];
        sxy += concurrency[i] * step_seconds[i];
    }
    const double den = n * sxx - sx * sx;
    if (!(std::fabs(den) > 0)) return PD_ERR_INVALID_ARG;
    *b = (n * sxy - sx * sy) / den;   // seconds per additional concurrent sequence
    *A = (sy - *b * sx) / n;          // fixed seconds per iteration
    return PD_OK;
}

}  // extern "C"
