"""The pins are only worth something if a plausible mistake in the oracle trips one of them.
Here mistakes are planted in copies of the oracle's C source (on the CPU, never in the CUDA path):
each mutated copy is compiled, swapped in for the real library, and at least one pin must fail."""
import ctypes
import os
import subprocess
import tempfile

import pytest

import oracle
import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(os.path.abspath(oracle.__file__)), "distrl_oracle.c")

PINS = [getattr(pins, n) for n in dir(pins) if n.startswith("test_")]

MUTATIONS = {
    "trace uses the step's own ratio instead of the next step's":
        ("double Delta = last ? delta : delta + gamma * c_next * Delta_next;",
         "double Delta = last ? delta : delta + gamma * c * Delta_next;"),
    "ratio not truncated at one":
        ("double c = lambda * fmin(1.0, rho);\n            double v_next", "double c = lambda * rho;\n            double v_next"),
    "ratio inverted (mu / pi)":
        ("double rho = exp(logp_pi[t] - logp_mu[t]);\n            double c", "double rho = exp(logp_mu[t] - logp_pi[t]);\n            double c"),
    "discount dropped from the bootstrap term":
        ("double delta = r[t] + gamma * v_next - V[t];", "double delta = r[t] + v_next - V[t];"),
    "sign of V(s_t) flipped":
        ("double delta = r[t] + gamma * v_next - V[t];", "double delta = r[t] + gamma * v_next + V[t];"),
    "bootstrap ignored":
        ("double v_next = last ? (boot ? boot[j] : 0.0) : V[t + 1];", "double v_next = last ? 0.0 : V[t + 1];"),
    "trajectory ends not recognised (only the buffer's last step counts as terminal)":
        ("int last = (t == off[j + 1] - 1);\n            double rho", "int last = (t == n - 1);\n            double rho"),
    "priority drops the entropy term":
        ("double p = w_td * fabs(td_delta[t]) + w_rho * fmin(rho, rho_clip) + w_ent * H;",
         "double p = w_td * fabs(td_delta[t]) + w_rho * fmin(rho, rho_clip);"),
    "priority uses signed delta":
        ("double p = w_td * fabs(td_delta[t]) + w_rho * fmin(rho, rho_clip) + w_ent * H;",
         "double p = w_td * td_delta[t] + w_rho * fmin(rho, rho_clip) + w_ent * H;"),
    "quantiser truncates instead of rounding to even":
        ("double rn = nearbyint(x);", "double rn = floor(x);"),
    "quantiser has no floor of one":
        ("q = (rn < 1.0) ? 1u : (uint32_t)rn;", "q = (uint32_t)rn;"),
    "sampler compares with >= (off by one mass unit)":
        ("if (run > y) { pick = i; break; }", "if (run >= y) { pick = i; break; }"),
    "importance weight exponent has the wrong sign":
        ("w_out[j] = pow((double)n * P, -beta);", "w_out[j] = pow((double)n * P, beta);"),
    "refresh: first duplicate wins instead of the last":
        ("for (int64_t j = 0; j < k; ++j) {\n        int64_t i = idx[j];", "for (int64_t j = k - 1; j >= 0; --j) {\n        int64_t i = idx[j];"),
    "Monte-Carlo return forgets the discount":
        ("g = r[t] + gamma * g;", "g = r[t] + g;"),
    "circular overwrite does not wrap":
        ("i = (i + 1) % n;", "i = (i + 1 < n) ? i + 1 : i;"),
    "actor coefficient: ratio inverted":
        ("double rho = exp(lp[i] - lm[i]);\n        coef[j]", "double rho = exp(lm[i] - lp[i]);\n        coef[j]"),
    "actor coefficient: importance-sampling weight dropped":
        ("coef[j] = (w ? w[j] : 1.0) * rho * adv[i];", "coef[j] = rho * adv[i];"),
    "actor coefficient: advantage read at the batch position instead of the drawn index":
        ("coef[j] = (w ? w[j] : 1.0) * rho * adv[i];", "coef[j] = (w ? w[j] : 1.0) * rho * adv[j];"),
    "filter keeps the low-scored trajectories instead of the high-scored ones":
        ("if (score[j] >= threshold) { ++kept; continue; }", "if (score[j] < threshold) { ++kept; continue; }"),
    "filter leaves a dropped trajectory's last transition in place":
        ("for (int64_t t = off[j]; t < off[j + 1]; ++t) q[t] = 0u;", "for (int64_t t = off[j]; t < off[j + 1] - 1; ++t) q[t] = 0u;"),
    "refresh drops the entropy term":
        ("double p = w_td * fabs(new_abs_delta[j]) + w_rho * fmin(rho, rho_clip) + w_ent * H;",
         "double p = w_td * fabs(new_abs_delta[j]) + w_rho * fmin(rho, rho_clip);"),
    "refresh: ratio inverted":
        ("double rho = exp(logp_pi[i] - logp_mu[i]);\n        double H", "double rho = exp(logp_mu[i] - logp_pi[i]);\n        double H"),
    "refresh: ratio not clipped":
        ("double p = w_td * fabs(new_abs_delta[j]) + w_rho * fmin(rho, rho_clip) + w_ent * H;",
         "double p = w_td * fabs(new_abs_delta[j]) + w_rho * rho + w_ent * H;"),
    "refresh: entropy fallback has the wrong sign":
        ("double H = entropy ? entropy[i] : -logp_pi[i];", "double H = entropy ? entropy[i] : logp_pi[i];"),
    "refresh: entropy read at the batch position instead of the refreshed index":
        ("double H = entropy ? entropy[i] : -logp_pi[i];", "double H = entropy ? entropy[j] : -logp_pi[i];"),
    "refresh: exponent alpha ignored":
        ("double mass = pow(p, alpha);\n        float mf", "double mass = p;\n        float mf"),
    "trajectory priority: entropy fallback has the wrong sign":
        ("sh += entropy ? entropy[t] : -logp_pi[t];", "sh += entropy ? entropy[t] : logp_pi[t];"),
    "trajectory priority: ratio not clipped":
        ("sr += fmin(exp(logp_pi[t] - logp_mu[t]), rho_clip);", "sr += exp(logp_pi[t] - logp_mu[t]);"),
    "trajectory priority: ratio inverted":
        ("sr += fmin(exp(logp_pi[t] - logp_mu[t]), rho_clip);", "sr += fmin(exp(logp_mu[t] - logp_pi[t]), rho_clip);"),
    "trajectory priority: sums instead of means":
        ("double p = w_td * (sd / (double)len) + w_rho * (sr / (double)len)", "double p = w_td * sd + w_rho * (sr / (double)len)"),
    "priority: entropy fallback has the wrong sign":
        ("double H = entropy ? entropy[t] : -logp_pi[t];", "double H = entropy ? entropy[t] : logp_pi[t];"),
    "priority: ratio not clipped":
        ("double p = w_td * fabs(td_delta[t]) + w_rho * fmin(rho, rho_clip) + w_ent * H;",
         "double p = w_td * fabs(td_delta[t]) + w_rho * rho + w_ent * H;"),
    "ring: a trajectory that does not fit at the end is squeezed in there instead of starting at slot 0":
        ("            h = 0;\n        }\n        /* every stored trajectory", "            h = n - T;\n        }\n        /* every stored trajectory"),
    "ring: the remainder of an evicted trajectory keeps its mass":
        ("for (int64_t t = s; t < e; ++t) { alive[t] = 0; q[t] = 0u; }", "for (int64_t t = s; t < e; ++t) { alive[t] = 0; }"),
    "ring: only the overwritten rows of an evicted trajectory die":
        ("    while (!start[s]) --s;             /* first slot of the trajectory that owns slot i */\n    while (e < n && !start[e]) ++e;",
         "    while (e < n && 0) ++e;"),
    "ring: what follows a new trajectory is not split off":
        ("if (h + T < n) start[h + T] = 1;", ";"),
    "ring: the slots retired at the end of the buffer keep their trajectories":
        ("for (int64_t i = h; i < n; ++i) ring_kill_trajectory_at(n, q, alive, start, i);\n            for (int64_t i = h; i < n; ++i) start[i] = (i == h);",
         "for (int64_t i = h; i < n; ++i) start[i] = (i == h);"),
    "ring: the write index does not come back to 0 after the last slot":
        ("*head = h % n;", "*head = h;"),
    "ring: the slots retired at the end are not counted, so a call may overwrite its own trajectories":
        ("if (h + T > n) { advance += n - h; h = 0; }", "if (h + T > n) { h = 0; }"),
    "ring: rows are taken from the start of the call's rows for every trajectory":
        ("field[f][h + i] = new_field[f][new_off[j] + i];", "field[f][h + i] = new_field[f][i];"),
    "stratified draws: the stratum index is not scaled to fixed point":
        ("unsigned __int128 x = ((unsigned __int128)(uint64_t)j << 64) + u[j];", "unsigned __int128 x = (unsigned __int128)(uint64_t)j + u[j];"),
    "trajectory range ends at its own start offset":
        ("end[j] = off[idx[j] + 1];", "end[j] = off[idx[j]];"),
}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_a_planted_mistake_trips_a_pin(name, monkeypatch):
    old, new = MUTATIONS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, "mutation site not found exactly once: " + name
    with tempfile.TemporaryDirectory() as d:
        src = os.path.join(d, "mutant.c")
        lib = os.path.join(d, "mutant.so")
        open(src, "w").write(text.replace(old, new))
        subprocess.check_call(["gcc", "-O1", "-std=c11", "-ffp-contract=off", "-shared", "-fPIC", "-o", lib, src, "-lm"])
        monkeypatch.setattr(oracle, "_lib", ctypes.CDLL(lib))
        tripped = []
        for pin in PINS:
            try:
                pin()
            except AssertionError:
                tripped.append(pin.__name__)
        assert tripped, "no pin noticed: " + name
