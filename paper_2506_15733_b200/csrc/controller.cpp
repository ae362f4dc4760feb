// Host-side controller of the SPECS loop (Algorithm 1 of the paper): per problem, which model
// drafts the next n candidate blocks, the append of the selected block, the dynamic switch
// (Step III, Section 2.3) and the stop at the target length.  The policies cover the paper's
// ablations (Section 4.3: only-small generation, random switching, draft start) and its two
// baselines (Section 4.1: beam search with a single model, RSD++).  Pure host logic: generation,
// scoring and selection are the caller's (the selection flags come from specs_subsample /
// specs_select / specs_beam_step); nothing here touches a GPU.
#include <new>
#include <vector>

#include "specs.h"

struct specs_controller {
    specs_policy policy;
    int32_t problems;
    std::vector<int32_t> gen;              // model that drafts the next step
    std::vector<int64_t> length, steps, target_steps, target_calls;
    std::vector<uint8_t> appended;         // whether the last advance() appended the problem's selected block

    bool done(int32_t p) const { return length[p] >= policy.target_len || steps[p] >= policy.max_steps; }
};

extern "C" {

int specs_controller_create(specs_controller** out, int32_t P, const specs_policy* policy) {
    if (!out || !policy) return SPECS_ERR_NULL;
    *out = nullptr;
    if (P < 0 || policy->policy < SPECS_POLICY_SPECS || policy->policy > SPECS_POLICY_RSD ||
        policy->target_len < 0 || policy->max_steps < 0 || !(policy->p_target >= 0.0f && policy->p_target <= 1.0f))
        return SPECS_ERR_SHAPE;
    specs_controller* c = new (std::nothrow) specs_controller();
    if (!c) return SPECS_ERR_CUDA;
    c->policy = *policy;
    c->problems = P;
    // Algorithm 1 begins with the target model; the draft-only, draft-start and RSD++ policies with the draft
    const bool draft_first = policy->policy == SPECS_POLICY_ONLY_DRAFT || policy->policy == SPECS_POLICY_DRAFT_START ||
                             policy->policy == SPECS_POLICY_RSD;
    c->gen.assign(P, draft_first ? SPECS_GEN_DRAFT : SPECS_GEN_TARGET);
    c->length.assign(P, 0);
    c->steps.assign(P, 0);
    c->target_steps.assign(P, 0);
    c->target_calls.assign(P, 0);
    c->appended.assign(P, 0);
    *out = c;
    return SPECS_OK;
}

int specs_controller_destroy(specs_controller* c) {
    delete c;
    return SPECS_OK;
}

int specs_controller_generators(const specs_controller* c, int32_t* h_gen) {
    if (!c || (!h_gen && c->problems > 0)) return SPECS_ERR_NULL;
    for (int32_t p = 0; p < c->problems; ++p) h_gen[p] = c->done(p) ? SPECS_GEN_DONE : c->gen[p];
    return SPECS_OK;
}

int specs_controller_advance(specs_controller* c, const int32_t* h_chosen, const uint8_t* h_flag,
                             const int64_t* h_chosen_len, const float* h_uniforms) {
    if (!c) return SPECS_ERR_NULL;
    if (c->problems == 0) return SPECS_OK;
    if (!h_chosen || !h_flag || !h_chosen_len) return SPECS_ERR_NULL;
    if (c->policy.policy == SPECS_POLICY_RANDOM && !h_uniforms) return SPECS_ERR_NULL;
    for (int32_t p = 0; p < c->problems; ++p)
        if (!c->done(p) && h_chosen[p] >= 0 && h_chosen_len[p] < 0) return SPECS_ERR_SHAPE;
    for (int32_t p = 0; p < c->problems; ++p) {
        c->appended[p] = 0;
        if (c->done(p)) continue;
        const int32_t g = c->gen[p];
        if (g == SPECS_GEN_TARGET) ++c->target_calls[p];
        if (c->policy.policy == SPECS_POLICY_RSD && g == SPECS_GEN_DRAFT && h_flag[p]) {
            c->gen[p] = SPECS_GEN_TARGET;          // the draft's best candidate is too weak: the target redoes the step
            continue;
        }
        if (h_chosen[p] >= 0) {                    // append the selected block
            c->length[p] += h_chosen_len[p];
            ++c->steps[p];
            c->appended[p] = 1;
            if (g == SPECS_GEN_TARGET) ++c->target_steps[p];
        }
        switch (c->policy.policy) {
            case SPECS_POLICY_SPECS:               // Step III: a high reward hands the next step to the draft
                if (h_flag[p]) c->gen[p] = SPECS_GEN_DRAFT;
                else if (!c->policy.sticky) c->gen[p] = SPECS_GEN_TARGET;
                break;
            case SPECS_POLICY_DRAFT_START:         // no candidate above tau: the target takes the next step
                if (h_flag[p]) c->gen[p] = SPECS_GEN_TARGET;
                else if (!c->policy.sticky) c->gen[p] = SPECS_GEN_DRAFT;
                break;
            case SPECS_POLICY_RANDOM:
                c->gen[p] = h_uniforms[p] < c->policy.p_target ? SPECS_GEN_TARGET : SPECS_GEN_DRAFT;
                break;
            case SPECS_POLICY_RSD:
                c->gen[p] = SPECS_GEN_DRAFT;
                break;
            default:                               // single-model policies never change
                break;
        }
    }
    return SPECS_OK;
}

int specs_controller_appended(const specs_controller* c, uint8_t* h_appended) {
    if (!c || (!h_appended && c->problems > 0)) return SPECS_ERR_NULL;
    for (int32_t p = 0; p < c->problems; ++p) h_appended[p] = c->appended[p];
    return SPECS_OK;
}

int specs_controller_stats(const specs_controller* c, int64_t* h_length, int64_t* h_steps, int64_t* h_target_steps,
                           int64_t* h_target_calls) {
    if (!c) return SPECS_ERR_NULL;
    for (int32_t p = 0; p < c->problems; ++p) {
        if (h_length) h_length[p] = c->length[p];
        if (h_steps) h_steps[p] = c->steps[p];
        if (h_target_steps) h_target_steps[p] = c->target_steps[p];
        if (h_target_calls) h_target_calls[p] = c->target_calls[p];
    }
    return SPECS_OK;
}

}  // extern "C"
