"""Sizing arithmetic: KV footprint (Eq. 1), offload benefit ratio (Eq. 2), working-set
scale (Eq. 5), pressure ratios (Section 3.2) and tier capacity in chunks (Section 4)."""
import math


def beta_rank(num_layers, head_dim, elem_bytes, kv_heads, tp=1):
    """Eq. 1: KV bytes per token on one rank = 2 L d s max(1, ceil(H_kv / TP))."""
    return 2 * num_layers * head_dim * elem_bytes * max(1, math.ceil(kv_heads / tp))


def tier_chunks(capacity_bytes, chunk_tokens, beta):
    """K_H = floor(C_H / (b * beta)) (Section 4, "Which writes a tier can decline")."""
    return capacity_bytes // (chunk_tokens * beta)


def working_set_bytes(active_pool, mean_prompt_tokens, beta):
    """Eq. 5: C_reuse ~ (A - 1) * N_bar * beta."""
    return (active_pool - 1) * mean_prompt_tokens * beta


def gamma_g(active_pool, mean_prompt_tokens, gpu_kv_tokens):
    """gamma_G = A * N_bar / K_G (Section 3.2)."""
    return active_pool * mean_prompt_tokens / gpu_kv_tokens


def gamma_h(working_set, host_capacity_bytes):
    """gamma_H = C_reuse / C_H (Section 3.2)."""
    return working_set / host_capacity_bytes


def load_time(n_tokens, beta, h2d_bytes_per_s, tau_load=0.0):
    """Eq. 2: T_load(n) = n * beta / B_H2D + tau_load."""
    return n_tokens * beta / h2d_bytes_per_s + tau_load


def obr(n_tokens, t_prefill_per_token, beta, h2d_bytes_per_s, tau_load=0.0):
    """Eq. 2: OBR(n) = 1 - T_load(n) / T_rec(n), T_rec(n) = n * t_pf."""
    return 1.0 - load_time(n_tokens, beta, h2d_bytes_per_s, tau_load) / (n_tokens * t_prefill_per_token)
