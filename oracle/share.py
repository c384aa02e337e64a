"""Test infrastructure only: the allocation statistic of Fig. 3 — how the Phase-B budget and the prompts split
over the Phase-A success count c (Sec. 4.1, paragraph on how the budget is reallocated).  Plain loops."""


def allocation_share(c, delta, G0: int):
    """(prompts[k], budget[k]) for k = 0..G0: number of prompts with c_i = k and the rollouts they received."""
    prompts = [0] * (G0 + 1)
    budget = [0] * (G0 + 1)
    for ci, di in zip(c, delta):
        ci = int(ci)
        if not 0 <= ci <= G0:
            raise ValueError("c outside [0, G0]")
        prompts[ci] += 1
        budget[ci] += int(di)
    return prompts, budget
