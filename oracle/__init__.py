"""Double-precision CPU oracle (test infrastructure; see svd_attention.py)."""
from .svd_attention import (  # noqa: F401
    hestenes_svd, sign_gauge, truncated_svd, factor_tokens, row_softmax,
    svd_attention_from_factors, svd_attention, softmax_attention,
    chain_attention, linear_attention, factored_exact_attention,
    householder_qr_basis, randomized_svd, max_rel_err_rows,
)
