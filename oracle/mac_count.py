"""Analytic MAC / activation-memory counts of the paper's resource-usage section.

TEST INFRASTRUCTURE ONLY.  Restates the dense Transformer-XL cost (Eq. "N_MAC^XL",
"N_mem^XL") and the SwitchHead cost (Eq. "N_MAC^SwitchHead") per layer per sequence.
T = sequence length, C = context multiple (C-1 cached chunks), M = d_model, D = d_head.

The SwitchHead equation as printed does not reproduce the SwitchHead rows of the paper's
result tables; `switchhead_macs_as_tabulated` (positional term counted once, plus the two
gate matmuls) does.  Both are kept; the tests pin each against the printed table values.
"""


def xl_macs(n_heads, T, D, M, C=2):
    return n_heads * (4 * T * D * M + 2 * C * T * T * D + 2 * C * T * D * M)


def xl_mem(n_heads, T, D, C=2):
    return n_heads * (4 * T * D + 2 * C * T * T + 2 * C * T * D)


def switchhead_macs_printed(n_heads, T, D, M, k, C=2):
    return n_heads * (2 * T * D * M + 2 * T * k * D * (M + 1) + 2 * C * T * T * D + 2 * C * T * D * M)


def switchhead_macs_as_tabulated(n_heads, T, D, M, k, E, C=2, n_gates=2):
    return n_heads * (2 * T * D * M + 2 * T * k * D * (M + 1) + 2 * C * T * T * D
                      + C * T * D * M + n_gates * T * M * E)


def switchhead_mem_as_tabulated(n_heads, T, D, C=2):
    return n_heads * (4 * T * D + 2 * C * T * T + C * T * D)


def forward_macs_no_positional(n_heads, T, D, M, k, E, causal_half=True):
    """MACs of the layer this repository computes (no XL cache, no positional projection):
    dense Q,K; k selected V and O experts with their weighted averages; both gates; attention."""
    attn = 2 * T * T * D
    if causal_half:
        attn //= 2
    return n_heads * (2 * T * D * M + 2 * T * k * D * (M + 1) + attn + 2 * T * M * E)
