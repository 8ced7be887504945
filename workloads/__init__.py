"""Seeded synthetic input generators (no attention arithmetic lives here)."""
