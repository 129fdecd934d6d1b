"""CPU oracle of the layout-operator chains (test infrastructure only)."""
