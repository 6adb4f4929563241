"""Float64 CPU oracle of the IPGS carve path (test infrastructure, never on the product path)."""
